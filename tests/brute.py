"""Exhaustive enumeration of the block-construction rule on tiny inputs.

The rule (Methods section; caption of the pseudocode figure): open a block, draw a random
sequence among those that still fit, repeat until nothing fits, pad, open the next block.
With 'random' read as uniform over the unused sequences that fit, the probability that the
next sequence has length l is count[l] / m (m = unused sequences that fit).  The outcome
(lengths in draw order, grouped in blocks) therefore has an exactly computable distribution.
"""
from fractions import Fraction
from functools import lru_cache
from itertools import combinations


def outcome_distribution(lengths, t_block, policy=0):
    """dict: outcome -> exact probability; outcome = tuple of blocks, block = tuple of lengths.
    policy 0: every unused sequence that fits is equally likely (P(length l) = count[l] / m);
    policy 1: every LENGTH that fits and is not exhausted is equally likely (P = 1 / #such lengths)."""
    start = tuple(sorted(lengths))

    @lru_cache(maxsize=None)
    def rec(left, room):
        # returns dict {tuple_of_blocks_from_here (first block partial): prob}
        if not left:
            return {((),): Fraction(1)}
        fit = [l for l in left if l <= room]
        out = {}
        if not fit:
            for tail, p in rec(left, t_block).items():
                out[((),) + tail] = out.get(((),) + tail, 0) + p
            return out
        m = len(fit)
        for l in sorted(set(fit)):
            pl = Fraction(fit.count(l), m) if policy == 0 else Fraction(1, len(set(fit)))
            rest = list(left)
            rest.remove(l)
            for tail, p in rec(tuple(rest), room - l).items():
                key = ((l,) + tail[0],) + tail[1:]
                out[key] = out.get(key, 0) + pl * p
        return out

    dist = rec(start, t_block)
    # a trailing empty block only appears when the recursion ends exactly at a block close
    clean = {}
    for k, p in dist.items():
        kk = tuple(b for b in k if b)
        clean[kk] = clean.get(kk, 0) + p
    assert sum(clean.values()) == 1
    return clean


def min_blocks(lengths, t_block):
    """Smallest number of blocks any assignment can reach (exhaustive)."""
    items = sorted(lengths, reverse=True)
    best = [len(items)]

    def rec(i, bins):
        if len(bins) >= best[0]:
            return
        if i == len(items):
            best[0] = len(bins)
            return
        seen = set()
        for j in range(len(bins)):
            if bins[j] + items[i] <= t_block and bins[j] not in seen:
                seen.add(bins[j])
                bins[j] += items[i]
                rec(i + 1, bins)
                bins[j] -= items[i]
        bins.append(items[i])
        rec(i + 1, bins)
        bins.pop()

    rec(0, [])
    return best[0]


def outcome_of_plan(lengths, n_blocks, seg_seq, block_seg_begin):
    return tuple(tuple(int(lengths[s]) for s in seg_seq[block_seg_begin[b]:block_seg_begin[b + 1]])
                 for b in range(n_blocks))
