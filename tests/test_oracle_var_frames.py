"""Pins for the oracle's per-sample frame sizes (byte_offsets, pack_var, unpack_var); no GPU."""
import numpy as np
import pytest

from oracle import bload_oracle as O


def _case(n, tb, seed, fmax):
    rng = np.random.default_rng(seed)
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    F = rng.integers(1, fmax + 1, size=n).astype(np.int32)
    return O.plan(T, tb, seed), T, F, rng


def test_byte_offsets_are_the_cumulative_sum_of_sequence_sizes():
    rng = np.random.default_rng(1)
    T = rng.integers(1, 5000, size=3000).astype(np.int32)
    F = rng.integers(1, 1 << 20, size=3000).astype(np.int32)
    want = np.concatenate([[0], np.cumsum(T.astype(np.int64) * F.astype(np.int64))])
    assert int(want[-1]) > 1 << 32
    assert np.array_equal(O.byte_offsets(T, F), want)


@pytest.mark.parametrize("fb", [1, 5, 16, 48])
def test_equal_frame_sizes_reduce_to_plain_pack_and_unpack(fb):
    p, T, _, rng = _case(120, 30, 3 + fb, 1)
    F = np.full(p.n, fb, np.int32)
    store = rng.integers(0, 256, size=p.sum_t * fb, dtype=np.uint8)
    nb = p.n_blocks + 1
    assert np.array_equal(O.pack_var(p, store, F, fb, 0, nb, 0x21), O.pack(p, store, fb, 0, nb, 0x21))
    dense_out = rng.integers(0, 256, size=nb * p.t_block * fb, dtype=np.uint8)
    a = np.full(p.sum_t * fb, 7, np.uint8); b = a.copy()
    O.unpack_var(p, dense_out, F, fb, 0, nb, a)
    O.unpack(p, dense_out, fb, 0, nb, b)
    assert np.array_equal(a, b)


@pytest.mark.parametrize("n,tb,fmax", [(8, 6, 9), (60, 20, 40), (150, 64, 7)])
def test_pack_var_places_every_image_at_the_start_of_its_slot(n, tb, fmax):
    # frames are H_i x W_i images (row major); a slot is a canvas of fmax bytes
    rng = np.random.default_rng(n)
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    H = rng.integers(1, 4, size=n); Wd = rng.integers(1, fmax // 3 + 1, size=n)
    F = (H * Wd).astype(np.int32)
    p = O.plan(T, tb, 50 + n)
    videos = [rng.integers(0, 256, size=(int(T[i]), int(H[i]), int(Wd[i])), dtype=np.uint8) for i in range(n)]
    store = np.concatenate([v.reshape(-1) for v in videos])
    nb = p.n_blocks + 1
    got = O.pack_var(p, store, F, fmax, 0, nb, 0xEE)
    seq_id, pos, _, valid = O.metadata(p, 0, nb)
    for q in range(nb):
        for s in range(tb):
            if valid[q, s]:
                img = videos[seq_id[q, s]][pos[q, s]].reshape(-1)
                assert np.array_equal(got[q, s, :img.size], img)
                assert np.all(got[q, s, img.size:] == 0xEE)
            else:
                assert np.all(got[q, s] == 0xEE)
    # sub-range
    assert np.array_equal(O.pack_var(p, store, F, fmax, 1, 2, 0xEE), got[1:3])
    # round trip: cropping every slot back gives the store, and touches nothing else
    back = np.full(store.size, 0x99, np.uint8)
    O.unpack_var(p, got, F, fmax, 0, nb, back)
    assert np.array_equal(back, store)
    part = np.full(store.size, 0x99, np.uint8)
    O.unpack_var(p, got[:1], F, fmax, 0, 1, part)
    boff = O.byte_offsets(T, F)
    inside = np.zeros(store.size, bool)
    for k in range(p.block_seg_begin[0], p.block_seg_begin[1]):
        i = int(p.seg_seq[k]); inside[boff[i]:boff[i + 1]] = True
    assert np.array_equal(part[inside], store[inside]) and np.all(part[~inside] == 0x99)


@pytest.mark.parametrize("n,tb,hmax,wmax", [(8, 6, 3, 5), (50, 20, 6, 16), (120, 40, 4, 9)])
def test_pack_var2d_places_every_image_in_the_top_left_corner_of_its_canvas(n, tb, hmax, wmax):
    rng = np.random.default_rng(n + hmax)
    T = rng.integers(1, tb + 1, size=n).astype(np.int32)
    H = rng.integers(1, hmax + 1, size=n).astype(np.int32)
    Wd = rng.integers(1, wmax + 1, size=n).astype(np.int32)
    p = O.plan(T, tb, 70 + n)
    videos = [rng.integers(0, 256, size=(int(T[i]), int(H[i]), int(Wd[i])), dtype=np.uint8) for i in range(n)]
    store = np.concatenate([v.reshape(-1) for v in videos])
    assert np.array_equal(O.byte_offsets2d(T, H, Wd),
                          np.concatenate([[0], np.cumsum(T.astype(np.int64) * H * Wd)]))
    nb = p.n_blocks + 1
    stride = wmax + 3
    got = O.pack_var2d(p, store, H, Wd, hmax, stride, 0, nb, 0xEE)
    seq_id, pos, _, valid = O.metadata(p, 0, nb)
    want = np.full((nb, tb, hmax, stride), 0xEE, np.uint8)
    for q in range(nb):
        for s in range(tb):
            if valid[q, s]:
                img = videos[seq_id[q, s]][pos[q, s]]
                want[q, s, :img.shape[0], :img.shape[1]] = img
    assert np.array_equal(got, want)
    assert np.array_equal(O.pack_var2d(p, store, H, Wd, hmax, stride, 1, 2, 0xEE), want[1:3])
    back = np.full(store.size, 0x99, np.uint8)
    O.unpack_var2d(p, got, H, Wd, hmax, stride, 0, nb, back)
    assert np.array_equal(back, store)


def test_one_row_per_image_reduces_to_pack_var():
    p, T, F, rng = _case(90, 25, 4, 30)
    store = rng.integers(0, 256, size=int(O.byte_offsets(T, F)[-1]), dtype=np.uint8)
    ones = np.ones(p.n, np.int32)
    nb = p.n_blocks + 1
    a = O.pack_var2d(p, store, ones, F, 1, 33, 0, nb, 5).reshape(nb, p.t_block, 33)
    assert np.array_equal(a, O.pack_var(p, store, F, 33, 0, nb, 5))
