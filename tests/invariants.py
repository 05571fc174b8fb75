"""Independent validity checker for a block plan (numpy only).

It knows nothing about how a plan was produced.  It checks what the paper fixes
for ANY output of the block-construction rule:
  I1  no frame dropped or duplicated: the segment list is a permutation of the sequences
  I2  a sequence occupies one contiguous run of one block, in frame order
  I3  no block holds more than t_block frames; blocks are filled front to back
  I4  a start-table entry (reset flag) sits at the first slot of every segment and nowhere else
  I5  a block is closed only when nothing that is left fits (maximality)
  I6  pad slots carry no sequence (checked on metadata / packed bytes by the callers)
"""
import numpy as np


class PlanError(AssertionError):
    pass


def _req(cond, msg):
    if not cond:
        raise PlanError(msg)


def check_plan(lengths, t_block, n_blocks, offsets, seg_seq, seg_block, seg_start, block_seg_begin,
               block_fill, seq_block, seq_start, maximal=True):
    """maximal=False skips I5, which belongs to the paper's rule (a block is closed only when nothing that is
    left fits) and does not hold for strategies that keep several blocks open."""
    T = np.asarray(lengths, dtype=np.int64)
    n = T.size
    seg_seq = np.asarray(seg_seq)[:n].astype(np.int64)
    seg_block = np.asarray(seg_block)[:n].astype(np.int64)
    seg_start = np.asarray(seg_start)[:n].astype(np.int64)
    bsb = np.asarray(block_seg_begin)[: n_blocks + 1].astype(np.int64)
    fill = np.asarray(block_fill)[:n_blocks].astype(np.int64)
    # ragged offsets
    _req(np.array_equal(np.asarray(offsets)[: n + 1], np.concatenate([[0], np.cumsum(T)])), "offsets")
    # I1
    _req(np.array_equal(np.sort(seg_seq), np.arange(n)), "I1: segment list is not a permutation")
    # CSR shape
    _req(n_blocks >= 1 and bsb[0] == 0 and bsb[-1] == n, "CSR ends")
    _req(np.all(np.diff(bsb) >= 1), "every block holds at least one sequence")
    _req(np.array_equal(seg_block, np.repeat(np.arange(n_blocks), np.diff(bsb))), "seg_block vs CSR")
    seg_len = T[seg_seq]
    # I2/I3: segments of a block are laid end to end from slot 0
    csum = np.cumsum(seg_len) - seg_len               # exclusive over all draws
    block_base = csum[bsb[:-1]]
    _req(np.array_equal(seg_start, csum - np.repeat(block_base, np.diff(bsb))), "I2: seg_start is not end-to-end")
    ends = np.add.reduceat(seg_len, bsb[:-1])
    _req(np.array_equal(fill, ends), "block_fill")
    _req(np.all(fill <= t_block) and np.all(fill >= 1), "I3: block over-full or empty")
    # I4 (table level): slot 0 of each block starts a segment
    _req(np.all(seg_start[bsb[:-1]] == 0), "I4: block does not begin with a sequence start")
    # inverse tables
    _req(np.array_equal(np.asarray(seq_block)[:n][seg_seq], seg_block), "seq_block")
    _req(np.array_equal(np.asarray(seq_start)[:n][seg_seq], seg_start), "seq_start")
    # I5: everything placed after block b was too long for the room left in b
    min_len_block = np.minimum.reduceat(seg_len, bsb[:-1])
    suffix_min = np.minimum.accumulate(min_len_block[::-1])[::-1]
    if n_blocks > 1 and maximal:
        _req(np.all(suffix_min[1:] > t_block - fill[:-1]), "I5: a later sequence would have fitted")
        _req(np.all(fill[:-1] + fill[1:] > t_block), "I5': adjacent blocks could merge")
    s = int(T.sum())
    _req(-(-s // t_block) <= n_blocks, "fewer blocks than the volume bound")
    if maximal:
        _req(n_blocks < 2 * s / t_block + 1, "I5'': too many blocks")
    return True


def slot_maps(lengths, t_block, n_blocks, seg_seq, seg_start, block_seg_begin, block_begin, block_count):
    """Per-slot metadata derived from the tables with numpy only (an independent route:
    built slot by slot from 'which segment covers slot s', not by walking segments)."""
    T = np.asarray(lengths, dtype=np.int64)
    seq_id = np.full((block_count, t_block), -1, np.int32)
    pos = np.full((block_count, t_block), -1, np.int32)
    reset = np.zeros((block_count, t_block), np.uint8)
    valid = np.zeros((block_count, t_block), np.uint8)
    slots = np.arange(t_block)
    for q in range(block_count):
        b = block_begin + q
        if b >= n_blocks:
            continue
        k0, k1 = int(block_seg_begin[b]), int(block_seg_begin[b + 1])
        st = np.asarray(seg_start[k0:k1], dtype=np.int64)
        ids = np.asarray(seg_seq[k0:k1], dtype=np.int64)
        which = np.searchsorted(st, slots, side="right") - 1        # covering segment
        inside = slots < st[which] + T[ids[which]]
        seq_id[q, inside] = ids[which][inside]
        pos[q, inside] = (slots - st[which])[inside]
        valid[q, inside] = 1
        reset[q, st] = 1
    return seq_id, pos, reset, valid
