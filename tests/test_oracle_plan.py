"""Pins for the oracle's block construction (no GPU)."""
import itertools

import numpy as np
import pytest
from scipy.stats import chi2

import brute
import invariants
from oracle import bload_oracle as O
from paper_2310_10879_b200 import workloads as W


def _check(p):
    assert p.status == 0
    invariants.check_plan(p.lengths, p.t_block, p.n_blocks, p.offsets, p.seg_seq, p.seg_block, p.seg_start,
                          p.block_seg_begin, p.block_fill, p.seq_block, p.seq_start)


def _golden(name):
    import os
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                out[k] = [int(x) for x in v]
    return out


def test_ldict_order_is_sorted_by_length_then_key_then_id():
    # a block long enough for everything and all lengths equal: the draw order IS the L_dict order
    n = 500
    T = np.full(n, 3, np.int32)
    for seed in (0, 9, 2**40 + 1):
        p = O.plan(T, 3 * n, seed)
        _check(p)
        want = sorted(range(n), key=lambda i: (O.seq_key(seed, i), i))
        assert list(p.seg_seq) == want and p.n_blocks == 1
    # ties on the key fall back to the id: force them by construction (same key for all is not
    # reachable through the hash, so check the comparator through two lengths instead)
    T = np.array([5, 2, 5, 2, 2], np.int32)
    p = O.plan(T, 16, 3)
    _check(p)
    for l in (2, 5):
        got = [int(s) for s in p.seg_seq if T[s] == l]
        assert got == sorted(got, key=lambda i: (O.seq_key(3, i), i))


def test_toy_dataset_of_the_paper_all_completions():
    g = _golden("paper_toy_dataset.txt")
    fixed, lo, hi = g["fixed_lengths"], g["t_min"][0], g["t_max"][0]
    completions = list(itertools.combinations_with_replacement(range(lo, hi + 1), g["n_videos"][0] - len(fixed)))
    assert len(completions) == 70
    for extra in completions:
        T = np.array(sorted(fixed + list(extra)), np.int32)
        dist = brute.outcome_distribution([int(x) for x in T], hi)
        opt = brute.min_blocks([int(x) for x in T], hi)
        for seed in range(25):
            p = O.plan(T, hi, seed)
            _check(p)
            assert brute.outcome_of_plan(T, p.n_blocks, p.seg_seq, p.block_seg_begin) in dist
            assert opt <= p.n_blocks <= max(len(k) for k in dist)
            s = O.stats(p.n, p.sum_t, p.t_max, p.t_block, p.n_blocks)
            assert s["pad_naive_tmax"] == 8 * 6 - int(T.sum())
            assert s["pad_packed"] == p.n_blocks * 6 - int(T.sum())


def test_toy_stand_in_counts():
    T = W.TOY8_LENGTHS
    assert int(T.sum()) == 31
    for seed in range(50):
        p = O.plan(T, W.TOY8_T_BLOCK, seed)
        _check(p)
        assert p.n_blocks >= 6
        s = O.stats(p.n, p.sum_t, p.t_max, p.t_block, p.n_blocks)
        assert s["pad_naive_tmax"] == 17 and s["pad_packed"] == 6 * p.n_blocks - 31


@pytest.mark.parametrize("lengths,t_block", [
    ([2, 2, 3, 3, 4, 5, 6, 6], 6),
    ([1, 1, 2, 3, 5], 5),
    ([4, 4, 3, 3, 2, 2, 1], 7),
    ([1, 2, 3, 4, 5, 6], 9),
])
def test_outcome_frequencies_match_exact_probabilities(lengths, t_block):
    """Over 10,000 fixed seeds the draw-order outcomes stay inside the reachable set of the rule and
    their frequencies agree with the exact probabilities prod(count[l]/m) (chi-square, fixed seeds)."""
    T = np.array(lengths, np.int32)
    dist = brute.outcome_distribution(lengths, t_block)
    n_seeds = 10000
    seen = {}
    for seed in range(n_seeds):
        p = O.plan(T, t_block, seed)
        k = brute.outcome_of_plan(T, p.n_blocks, p.seg_seq, p.block_seg_begin)
        assert k in dist, k
        seen[k] = seen.get(k, 0) + 1
    keys = sorted(dist, key=lambda k: -dist[k])
    exp = np.array([float(dist[k]) * n_seeds for k in keys])
    obs = np.array([seen.get(k, 0) for k in keys], dtype=float)
    big = exp >= 5
    e = np.append(exp[big], exp[~big].sum()) if (~big).any() else exp
    o = np.append(obs[big], obs[~big].sum()) if (~big).any() else obs
    keep = e > 0
    stat = float(((o[keep] - e[keep]) ** 2 / e[keep]).sum())
    assert stat < chi2.ppf(0.9999, keep.sum() - 1), (stat, keep.sum())
    # every outcome with a fair chance was actually seen: the rule is not a deterministic heuristic
    assert all(seen.get(k, 0) > 0 for k in keys if dist[k] * n_seeds >= 30)


def test_each_fitting_sequence_is_equally_likely():
    """'Randomly sampled sequences': the first draw is uniform over all N sequences when all fit, and
    with equal lengths the whole draw order is a uniform permutation."""
    T = np.array([2, 2, 3, 3, 4, 5, 6, 6], np.int32)
    first = np.zeros(8)
    n_seeds = 16000
    for seed in range(n_seeds):
        first[O.plan(T, 6, seed).seg_seq[0]] += 1
    stat = float(((first - n_seeds / 8) ** 2 / (n_seeds / 8)).sum())
    assert stat < chi2.ppf(0.9999, 7)
    T = np.full(4, 2, np.int32)
    perms = {}
    for seed in range(12000):
        k = tuple(int(x) for x in O.plan(T, 8, seed).seg_seq)
        perms[k] = perms.get(k, 0) + 1
    assert len(perms) == 24
    obs = np.array(list(perms.values()), float)
    assert float(((obs - 500.0) ** 2 / 500.0).sum()) < chi2.ppf(0.9999, 23)


def test_second_draw_conditional_distribution():
    """After a first draw of length a in a block of 6, the second draw is uniform over the unused
    sequences with T <= 6 - a (checked id by id, pooled over seeds)."""
    T = np.array([1, 1, 2, 2, 3, 3, 4, 5], np.int32)
    tb = 6
    table = {}
    for seed in range(30000):
        p = O.plan(T, tb, seed)
        a = int(p.seg_seq[0])
        if p.block_seg_begin[1] >= 2:
            table.setdefault(a, {}).setdefault(int(p.seg_seq[1]), 0)
            table[a][int(p.seg_seq[1])] += 1
    for a, row in table.items():
        room = tb - T[a]
        fits = [i for i in range(8) if i != a and T[i] <= room]
        assert set(row) <= set(fits)
        tot = sum(row.values())
        if tot >= 200 and len(fits) > 1:
            obs = np.array([row.get(i, 0) for i in fits], float)
            e = tot / len(fits)
            assert float(((obs - e) ** 2 / e).sum()) < chi2.ppf(0.9999, len(fits) - 1), (a, row)


def test_random_small_cases_stay_in_reachable_set():
    rng = np.random.default_rng(11)
    for _ in range(60):
        n = int(rng.integers(1, 8))
        tb = int(rng.integers(1, 10))
        T = rng.integers(1, tb + 1, size=n).astype(np.int32)
        dist = brute.outcome_distribution([int(x) for x in T], tb)
        opt = brute.min_blocks([int(x) for x in T], tb)
        for seed in range(20):
            p = O.plan(T, tb, seed)
            _check(p)
            assert brute.outcome_of_plan(T, p.n_blocks, p.seg_seq, p.block_seg_begin) in dist
            assert p.n_blocks >= opt


@pytest.mark.parametrize("name", ["toy_video", "features_fp16", "raw_frames", "heavy_tail_bf16",
                                  "video_dataset_shape"])
def test_invariants_on_workloads(name):
    w = W.WORKLOADS[name]
    T = W.lengths(w)
    p = O.plan(T, w.t_block, seed=w.seed)
    _check(p)
    assert p.sum_t == int(T.sum()) and p.t_max == int(T.max())
    assert p.max_segs_per_block == int(np.diff(p.block_seg_begin).max())


def test_invariants_on_token_workload_full_size():
    w = W.WORKLOADS["tokens"]
    T = W.lengths(w)
    p = O.plan(T, w.t_block, seed=w.seed)
    _check(p)


def test_degenerate_cases():
    # one sequence; all sequences as long as the block; all of length one; block of one slot
    p = O.plan(np.array([5], np.int32), 9, 1); _check(p); assert p.n_blocks == 1 and p.block_fill[0] == 5
    p = O.plan(np.full(17, 9, np.int32), 9, 1); _check(p); assert p.n_blocks == 17
    p = O.plan(np.ones(100, np.int32), 8, 1); _check(p); assert p.n_blocks == 13 and p.block_fill[-1] == 4
    p = O.plan(np.ones(5, np.int32), 1, 1); _check(p); assert p.n_blocks == 5
    # different seeds give different plans, equal seeds equal plans
    T = W.lengths(W.WORKLOADS["features_fp16"])
    a, b, c = O.plan(T, 1000, 1), O.plan(T, 1000, 1), O.plan(T, 1000, 2)
    assert np.array_equal(a.seg_seq, b.seg_seq) and a.checksum == b.checksum
    assert not np.array_equal(a.seg_seq, c.seg_seq) and a.checksum != c.checksum


def test_bad_inputs_are_rejected():
    p = O.plan(np.array([3, 0, 2], np.int32), 4, 0)
    assert p.status != 0 and p.first_bad == 1
    p = O.plan(np.array([3, 4, 5, 2], np.int32), 4, 0)
    assert p.status != 0 and p.first_bad == 2
    p = O.plan(np.array([3, -1], np.int32), 4, 0)
    assert p.status != 0 and p.first_bad == 1
    assert O.plan(np.array([1], np.int32), 0, 0).status != 0
    assert O.plan(np.array([], np.int32), 4, 0).status != 0
    assert O.plan(np.array([1], np.int32), 4, 0, policy=7).status != 0
    assert O.plan(np.array([1], np.int32), 4, 0, policy=1).status == 0


def test_checker_rejects_planted_mistakes():
    """The validity checker must bite: corrupt a correct plan in the ways an implementation could go wrong."""
    T = W.lengths(W.WORKLOADS["features_fp16"])
    p = O.plan(T, 1000, 3)
    args = dict(lengths=p.lengths, t_block=p.t_block, n_blocks=p.n_blocks, offsets=p.offsets, seg_seq=p.seg_seq,
                seg_block=p.seg_block, seg_start=p.seg_start, block_seg_begin=p.block_seg_begin,
                block_fill=p.block_fill, seq_block=p.seq_block, seq_start=p.seq_start)
    invariants.check_plan(**args)

    def broken(**kw):
        a = dict(args); a.update(kw)
        with pytest.raises(invariants.PlanError):
            invariants.check_plan(**a)

    x = p.seg_seq.copy(); x[5] = x[6]; broken(seg_seq=x)                     # a sequence dropped, one duplicated
    x = p.seg_start.copy(); x[1] += 1; broken(seg_start=x)                    # gap inside a block
    x = p.block_fill.copy(); x[0] -= 1; broken(block_fill=x)
    x = p.offsets.copy(); x[10] += 1; broken(offsets=x)
    x = p.seq_start.copy(); x[int(p.seg_seq[1])] += 1; broken(seq_start=x)
    # close the first block one draw early: the moved sequence would have fitted -> maximality
    bsb = p.block_seg_begin.copy(); bsb[1] -= 1
    sb = np.repeat(np.arange(p.n_blocks), np.diff(bsb)).astype(np.int32)
    Ts = p.lengths[p.seg_seq].astype(np.int64)
    st = (np.cumsum(Ts) - Ts); st = (st - np.repeat(st[bsb[:-1]], np.diff(bsb))).astype(np.int32)
    fill = np.add.reduceat(Ts, bsb[:-1]).astype(np.int32)
    sblk = np.empty_like(p.seq_block); sblk[p.seg_seq] = sb
    sst = np.empty_like(p.seq_start); sst[p.seg_seq] = st
    if fill.max() <= p.t_block:
        broken(block_seg_begin=bsb, seg_block=sb, seg_start=st, block_fill=fill, seq_block=sblk, seq_start=sst)


# ---- policy 1: the other reading of "a random entry of L_dict": a random KEY (length) that fits ----

@pytest.mark.parametrize("lengths,t_block", [
    ([2, 2, 2, 2, 3, 6, 6, 6], 6),
    ([1, 1, 1, 1, 1, 4, 5], 5),
    ([4, 3, 3, 3, 2, 1, 1, 1], 7),
])
def test_policy1_outcome_frequencies_match_uniform_over_lengths(lengths, t_block):
    T = np.array(lengths, np.int32)
    dist = brute.outcome_distribution(lengths, t_block, policy=1)
    other = brute.outcome_distribution(lengths, t_block, policy=0)
    tv = 0.5 * sum(abs(float(dist.get(k, 0)) - float(other.get(k, 0))) for k in set(dist) | set(other))
    assert tv > 0.05                                     # the two readings really differ on this input
    n_seeds = 10000
    seen = {}
    for seed in range(n_seeds):
        p = O.plan(T, t_block, seed, policy=1)
        _check(p)
        k = brute.outcome_of_plan(T, p.n_blocks, p.seg_seq, p.block_seg_begin)
        assert k in dist, k
        seen[k] = seen.get(k, 0) + 1
    keys = sorted(dist, key=lambda k: -dist[k])
    exp = np.array([float(dist[k]) * n_seeds for k in keys])
    obs = np.array([seen.get(k, 0) for k in keys], dtype=float)
    big = exp >= 5
    e = np.append(exp[big], exp[~big].sum()) if (~big).any() else exp
    o = np.append(obs[big], obs[~big].sum()) if (~big).any() else obs
    keep = e > 0
    stat = float(((o[keep] - e[keep]) ** 2 / e[keep]).sum())
    assert stat < chi2.ppf(0.9999, keep.sum() - 1), (stat, keep.sum())


def test_policy1_first_draw_is_uniform_over_lengths_not_sequences():
    T = np.array([1] * 9 + [2], np.int32)        # nine sequences of length 1, one of length 2
    hits = sum(int(T[O.plan(T, 4, seed, policy=1).seg_seq[0]] == 2) for seed in range(4000))
    assert 1800 < hits < 2200                     # 1/2 under policy 1 (it would be 1/10 under policy 0)
    hits0 = sum(int(T[O.plan(T, 4, seed, policy=0).seg_seq[0]] == 2) for seed in range(4000))
    assert 300 < hits0 < 500


@pytest.mark.parametrize("name", ["toy_video", "features_fp16", "heavy_tail_bf16", "video_dataset_shape"])
def test_policy1_invariants_on_workloads(name):
    w = W.WORKLOADS[name]
    T = W.lengths(w)
    p = O.plan(T, w.t_block, seed=w.seed, policy=1)
    _check(p)
    q = O.plan(T, w.t_block, seed=w.seed, policy=0)
    assert not np.array_equal(p.seg_seq, q.seg_seq)


def test_policy1_random_small_cases_stay_in_reachable_set():
    rng = np.random.default_rng(12)
    for _ in range(40):
        n = int(rng.integers(1, 8)); tb = int(rng.integers(1, 10))
        T = rng.integers(1, tb + 1, size=n).astype(np.int32)
        dist = brute.outcome_distribution([int(x) for x in T], tb, policy=1)
        for seed in range(15):
            p = O.plan(T, tb, seed, policy=1)
            _check(p)
            assert brute.outcome_of_plan(T, p.n_blocks, p.seg_seq, p.block_seg_begin) in dist


# ---- the plan digest, recomputed with Python integers ----

def _digest_with_python_integers(seg_block, seg_start, seg_seq):
    """Wrapping 64-bit sum, over the segments, of the 64-bit finaliser of MurmurHash3 (Appleby's public-domain
    fmix64: xor-shift 33, multiply, xor-shift 33, multiply, xor-shift 33) applied to
    (block << 32 | start) * golden-ratio constant + sequence.  Arbitrary-precision integers masked to 64 bits."""
    M = (1 << 64) - 1
    total = 0
    for b, s, q in zip(seg_block.tolist(), seg_start.tolist(), seg_seq.tolist()):
        k = ((((b & 0xFFFFFFFF) << 32) | (s & 0xFFFFFFFF)) * 0x9E3779B97F4A7C15 + (q & 0xFFFFFFFF)) & M
        k ^= k >> 33
        k = (k * 0xFF51AFD7ED558CCD) & M
        k ^= k >> 33
        k = (k * 0xC4CEB9FE1A85EC53) & M
        k ^= k >> 33
        total = (total + k) & M
    return total


@pytest.mark.parametrize("policy", [0, 1, 2])
def test_checksum_equals_a_big_integer_recomputation(policy):
    for name in ("toy_video", "features_fp16", "video_dataset_shape"):
        w = W.WORKLOADS[name]
        p = O.plan(W.lengths(w), w.t_block, seed=w.seed, policy=policy)
        assert p.checksum == _digest_with_python_integers(p.seg_block, p.seg_start, p.seg_seq), name


def test_checksum_with_block_and_sequence_numbers_beyond_16_bits():
    # 70,000 sequences of 3 or 4 frames in blocks of 4: one sequence per block, so block and sequence numbers pass
    # 2^16 and a digest that truncated either of them, or swapped block and start, would differ
    rng = np.random.default_rng(7)
    T = rng.integers(3, 5, size=70000).astype(np.int32)
    p = O.plan(T, 4, seed=11)
    assert p.n_blocks == 70000 and int(p.seg_block.max()) >= 1 << 16 and int(p.seg_seq.max()) >= 1 << 16
    want = _digest_with_python_integers(p.seg_block, p.seg_start, p.seg_seq)
    assert p.checksum == want
    # the digest depends on each of the three fields, and not on the order of the segments
    perm = rng.permutation(T.size)
    assert _digest_with_python_integers(p.seg_block[perm], p.seg_start[perm], p.seg_seq[perm]) == want
    assert _digest_with_python_integers(p.seg_block[::-1].copy(), p.seg_start, p.seg_seq) != want
    assert _digest_with_python_integers(p.seg_start, p.seg_block, p.seg_seq) != want
    # a plan with non-zero start slots (several sequences per block)
    T2 = rng.integers(1, 9, size=3000).astype(np.int32)
    p2 = O.plan(T2, 16, seed=5)
    assert int(p2.seg_start.max()) > 0
    assert p2.checksum == _digest_with_python_integers(p2.seg_block, p2.seg_start, p2.seg_seq)
