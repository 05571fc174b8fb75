"""GPU parity of per-sample frame sizes (bload_var_offsets, bload_pack_var, bload_unpack_var), through the
C ABI, against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O

pytestmark = pytest.mark.gpu


def _setup(T, F, tb, seed):
    T = np.ascontiguousarray(T, np.int32); F = np.ascontiguousarray(F, np.int32)
    op = O.plan(T, tb, seed)
    plan = G.gpu_plan(T, tb, seed)
    assert plan.info.checksum == op.checksum
    d_T = torch.from_numpy(T).to(G.DEV); d_F = torch.from_numpy(F).to(G.DEV)
    boff, info = B.bload_var_offsets(d_T, d_F)
    want = O.byte_offsets(T, F)
    assert np.array_equal(boff[:T.size + 1].cpu().numpy(), want)
    assert (info.total_bytes, info.max_frame_bytes, info.first_bad_index) == (int(want[-1]), int(F.max()), -1)
    return op, plan, d_F, boff, int(want[-1])


def _parity(T, F, tb, seed, slot, pad=0x6B, ranges=None):
    op, plan, d_F, boff, total = _setup(T, F, tb, seed)
    g = torch.Generator(device=G.DEV); g.manual_seed(seed)
    store = torch.randint(0, 256, (total,), dtype=torch.uint8, device=G.DEV, generator=g)
    store_h = store.cpu().numpy()
    for b0, cnt in ranges or ((0, op.n_blocks + 2), (1, max(op.n_blocks - 1, 1))):
        dense = G.Guarded(cnt * tb * slot)
        B.bload_pack_var(plan, store, d_F, boff, slot, b0, cnt, dense.t, pad_byte=pad)
        torch.cuda.synchronize(); dense.check()
        d = G.first_diff(dense.t.cpu().numpy(), O.pack_var(op, store_h, F, slot, b0, cnt, pad))
        assert d is None, "pack_var slot=%d blocks [%d,+%d): %s" % (slot, b0, cnt, d)
        dense_out = torch.randint(0, 256, (cnt * tb * slot,), dtype=torch.uint8, device=G.DEV, generator=g)
        rag = G.Guarded(total, 0x5A)
        B.bload_unpack_var(plan, dense_out, d_F, boff, slot, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        want = np.full(total, 0x5A, np.uint8)
        O.unpack_var(op, dense_out.cpu().numpy(), F, slot, b0, cnt, want)
        d = G.first_diff(rag.t.cpu().numpy(), want)
        assert d is None, "unpack_var slot=%d blocks [%d,+%d): %s" % (slot, b0, cnt, d)
    # round trip on the GPU alone
    nb = op.n_blocks
    dense = torch.empty(nb * tb * slot, dtype=torch.uint8, device=G.DEV)
    back = torch.full((total,), 0x11, dtype=torch.uint8, device=G.DEV)
    B.bload_pack_var(plan, store, d_F, boff, slot, 0, nb, dense)
    B.bload_unpack_var(plan, dense, d_F, boff, slot, 0, nb, back)
    torch.cuda.synchronize()
    assert torch.equal(back, store)


@pytest.mark.parametrize("fmax", [1, 3, 4, 16, 37, 100, 1000, 5000, 40000])
def test_random_frame_sizes(fmax):
    rng = np.random.default_rng(fmax)
    tb = int(rng.integers(4, 60))
    n = int(rng.integers(2, 120))
    T = rng.integers(1, tb + 1, size=n)
    F = rng.integers(1, fmax + 1, size=n)
    _parity(T, F, tb, 7 + fmax, slot=fmax)
    _parity(T, F, tb, 8 + fmax, slot=fmax + int(rng.integers(1, 40)))  # slots larger than every frame


def test_images_of_different_sizes():
    # H_i x W_i x 3 uint8 images on a canvas of the largest size; t_block spans several 16 KB sub-tiles per slot and
    # several slots per sub-tile
    rng = np.random.default_rng(2)
    n, tb = 60, 24
    T = rng.integers(1, tb + 1, size=n)
    H = rng.integers(8, 97, size=n); Wd = rng.integers(8, 129, size=n)
    F = H * Wd * 3
    _parity(T, F, tb, 99, slot=96 * 128 * 3)


def test_equal_sizes_match_the_fixed_size_calls():
    rng = np.random.default_rng(5)
    tb, fb = 50, 4096
    T = rng.integers(1, tb + 1, size=200).astype(np.int32)
    F = np.full(T.size, fb, np.int32)
    op, plan, d_F, boff, total = _setup(T, F, tb, 3)
    store = torch.randint(0, 256, (total,), dtype=torch.uint8, device=G.DEV)
    nb = op.n_blocks + 1
    a = torch.empty(nb * tb * fb, dtype=torch.uint8, device=G.DEV); b = torch.empty_like(a)
    B.bload_pack_var(plan, store, d_F, boff, fb, 0, nb, a, pad_byte=9)
    B.bload_pack(plan, store, fb, 0, nb, dense=b, pad_byte=9)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


def test_var_offsets_large_and_bad_sizes():
    rng = np.random.default_rng(6)
    n = 300_000
    T = rng.integers(1, 4096, size=n).astype(np.int32)
    F = rng.integers(1, 1 << 18, size=n).astype(np.int32)
    d_T = torch.from_numpy(T).to(G.DEV); d_F = torch.from_numpy(F).to(G.DEV)
    boff, info = B.bload_var_offsets(d_T, d_F)
    want = O.byte_offsets(T, F)
    assert int(want[-1]) > 1 << 40
    assert np.array_equal(boff[:n + 1].cpu().numpy(), want) and info.max_frame_bytes == int(F.max())
    F[1234] = 0; F[200_000] = -5
    with pytest.raises(B.BloadError) as e:
        B.bload_var_offsets(d_T, torch.from_numpy(F).to(G.DEV))
    assert e.value.code == -2 and e.value.info.first_bad_index == 1234


def test_var_calls_reject_bad_arguments():
    T = np.array([3, 4, 5], np.int32); F = np.array([8, 16, 4], np.int32)
    op, plan, d_F, boff, total = _setup(T, F, 8, 1)
    buf = torch.zeros(1 << 12, dtype=torch.uint8, device=G.DEV)
    for args, code in (((buf, d_F, boff, 0, 0, 1, buf), -2), ((buf, d_F, boff, 16, -1, 1, buf), -2),
                       ((None, d_F, boff, 16, 0, 1, buf), -1), ((buf, None, boff, 16, 0, 1, buf), -1),
                       ((buf[4:], d_F, boff, 16, 0, 1, buf), -5)):
        with pytest.raises(B.BloadError) as e:
            B.bload_pack_var(plan, *args)
        assert e.value.code == code
        with pytest.raises(B.BloadError) as e:
            B.bload_unpack_var(plan, *args)
        assert e.value.code == code


def _parity2d(T, H, Wb, tb, seed, hmax, stride, pad=0x6B):
    T = np.ascontiguousarray(T, np.int32); H = np.ascontiguousarray(H, np.int32); Wb = np.ascontiguousarray(Wb, np.int32)
    op = O.plan(T, tb, seed)
    plan = G.gpu_plan(T, tb, seed)
    d_T, d_H, d_W = (torch.from_numpy(x).to(G.DEV) for x in (T, H, Wb))
    boff, info = B.bload_var_offsets2d(d_T, d_H, d_W)
    want_off = O.byte_offsets2d(T, H, Wb)
    assert np.array_equal(boff[:T.size + 1].cpu().numpy(), want_off)
    assert (info.total_bytes, info.max_frame_bytes, info.max_rows, info.first_bad_index) == \
        (int(want_off[-1]), int(Wb.max()), int(H.max()), -1)
    total = int(want_off[-1])
    g = torch.Generator(device=G.DEV); g.manual_seed(seed)
    store = torch.randint(0, 256, (total,), dtype=torch.uint8, device=G.DEV, generator=g)
    store_h = store.cpu().numpy()
    canvas = hmax * stride
    for b0, cnt in ((0, op.n_blocks + 2), (1, max(op.n_blocks - 1, 1))):
        dense = G.Guarded(cnt * tb * canvas)
        B.bload_pack_var2d(plan, store, d_H, d_W, boff, hmax, stride, b0, cnt, dense.t, pad_byte=pad)
        torch.cuda.synchronize(); dense.check()
        d = G.first_diff(dense.t.cpu().numpy(), O.pack_var2d(op, store_h, H, Wb, hmax, stride, b0, cnt, pad))
        assert d is None, "pack_var2d %dx%d blocks [%d,+%d): %s" % (hmax, stride, b0, cnt, d)
        dense_out = torch.randint(0, 256, (cnt * tb * canvas,), dtype=torch.uint8, device=G.DEV, generator=g)
        rag = G.Guarded(total, 0x5A)
        B.bload_unpack_var2d(plan, dense_out, d_H, d_W, boff, hmax, stride, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        want = np.full(total, 0x5A, np.uint8)
        O.unpack_var2d(op, dense_out.cpu().numpy(), H, Wb, hmax, stride, b0, cnt, want)
        d = G.first_diff(rag.t.cpu().numpy(), want)
        assert d is None, "unpack_var2d %dx%d blocks [%d,+%d): %s" % (hmax, stride, b0, cnt, d)


@pytest.mark.parametrize("hmax,wmax,extra", [(1, 7, 0), (3, 5, 2), (4, 16, 0), (7, 33, 5), (16, 100, 0), (40, 700, 4),
                                             (224, 672, 0)])
def test_images_on_canvases(hmax, wmax, extra):
    rng = np.random.default_rng(hmax * 1000 + wmax)
    tb = int(rng.integers(3, 30))
    n = int(rng.integers(2, 60))
    T = rng.integers(1, tb + 1, size=n)
    H = rng.integers(1, hmax + 1, size=n)
    Wb = rng.integers(1, wmax + 1, size=n)
    H[0], Wb[0] = hmax, wmax  # one image fills its canvas (when extra == 0): the contiguous path
    _parity2d(T, H, Wb, tb, 5 + hmax, hmax, wmax + extra)


def test_canvases_of_equal_images_match_the_fixed_size_pack():
    rng = np.random.default_rng(8)
    tb, h, wb = 30, 6, 48
    T = rng.integers(1, tb + 1, size=100).astype(np.int32)
    plan = G.gpu_plan(T, tb, 2)
    d_T = torch.from_numpy(T).to(G.DEV)
    d_H = torch.full((T.size,), h, dtype=torch.int32, device=G.DEV)
    d_W = torch.full((T.size,), wb, dtype=torch.int32, device=G.DEV)
    boff, info = B.bload_var_offsets2d(d_T, d_H, d_W)
    store = torch.randint(0, 256, (info.total_bytes,), dtype=torch.uint8, device=G.DEV)
    nb = plan.n_blocks + 1
    a = torch.empty(nb * tb * h * wb, dtype=torch.uint8, device=G.DEV); b = torch.empty_like(a)
    B.bload_pack_var2d(plan, store, d_H, d_W, boff, h, wb, 0, nb, a, pad_byte=3)
    B.bload_pack(plan, store, h * wb, 0, nb, dense=b, pad_byte=3)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


@pytest.mark.parametrize("unit,kmax,extra", [(16, 1, 0), (16, 9, 16), (64, 16, 0), (256, 16, 48), (1024, 4, 0), (1024, 40, 1024)])
def test_frame_sizes_that_are_multiples_of_16_bytes(unit, kmax, extra):
    """Frames and slots whose sizes are multiples of 16 bytes take the kernel's flat vector loop; a few sizes that are
    not are mixed in, so that one launch holds segments of both kinds."""
    rng = np.random.default_rng(unit + kmax)
    tb = int(rng.integers(4, 70))
    n = int(rng.integers(20, 200))
    T = rng.integers(1, tb + 1, size=n)
    F = rng.integers(1, kmax + 1, size=n) * unit
    F[-3:] = np.maximum(F[-3:] - 4, 4)           # the last sequences: word-aligned but not vector-aligned sizes and offsets
    _parity(T, F, tb, 21 + unit, slot=unit * kmax + extra)


@pytest.mark.parametrize("hmax,unit,kmax,extra", [(1, 16, 8, 16), (3, 16, 5, 0), (5, 32, 9, 32), (12, 128, 6, 0), (40, 16, 50, 16)])
def test_images_whose_rows_are_multiples_of_16_bytes(hmax, unit, kmax, extra):
    rng = np.random.default_rng(hmax * 100 + kmax)
    tb = int(rng.integers(3, 40))
    n = int(rng.integers(5, 80))
    T = rng.integers(1, tb + 1, size=n)
    H = rng.integers(1, hmax + 1, size=n)
    Wb = rng.integers(1, kmax + 1, size=n) * unit
    H[0], Wb[0] = hmax, kmax * unit
    Wb[-1] = max(4, Wb[-1] - 8)                  # the last sequence is off the vector path
    _parity2d(T, H, Wb, tb, 9 + hmax, hmax, kmax * unit + extra)
