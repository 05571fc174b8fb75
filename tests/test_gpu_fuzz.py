"""Randomised GPU parity: many small random problems (sizes, block lengths, frame sizes, policies, block ranges, pad
bytes), every one compared bit for bit with the oracle.  Seeds are fixed, so the cases are the same on every run; they
are drawn to hit every copy kernel (register path, staged pack, staged unpack of sub-ranges, ragged-tiled unpack)."""
import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O

pytestmark = pytest.mark.gpu


def _case(rng):
    tb = int(rng.choice([1, 2, 3, 7, 16, 33, 64, 100, 257, 1000, 4096]))
    n = int(rng.choice([1, 2, 5, 31, 64, 300, 2049, 6000]))
    shape = rng.choice(["uniform", "short", "long", "two"])
    if shape == "uniform":
        T = rng.integers(1, tb + 1, size=n)
    elif shape == "short":
        T = rng.integers(1, max(2, tb // 8 + 1), size=n)
    elif shape == "long":
        T = np.maximum(1, tb - rng.integers(0, max(1, tb // 4), size=n))
    else:
        T = rng.choice([1, tb], size=n)
    fb = int(rng.choice([1, 2, 3, 4, 4, 8, 12, 16, 20, 36, 64, 100, 256, 520, 1024, 4100]))
    T = T.astype(np.int32)
    while int(T.sum()) * fb > 48_000_000:      # keep every case small
        T = T[: max(1, T.size // 2)]
    return T, tb, fb, int(rng.integers(0, 3)), int(rng.integers(0, 1 << 62)), int(rng.integers(0, 256))


@pytest.mark.parametrize("chunk", range(6))
def test_random_problems(chunk):
    rng = np.random.default_rng(9000 + chunk)
    for _ in range(25):
        T, tb, fb, policy, seed, pad = _case(rng)
        op = O.plan(T, tb, seed, policy)
        plan = G.gpu_plan(T, tb, seed, policy=policy)
        G.assert_plan_equal(plan, op)
        store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=G.DEV)
        store_h = store.cpu().numpy()
        # a random block range (possibly reaching past the end) and the whole plan
        b0 = int(rng.integers(0, op.n_blocks)); cnt = int(rng.integers(1, op.n_blocks - b0 + 3))
        for lo, c in ((b0, cnt), (0, op.n_blocks)):
            res, dense = G.gpu_pack_all(plan, store, fb, lo, c, pad)
            assert np.array_equal(res["dense"], O.pack(op, store_h, fb, lo, c, pad)), (T.size, tb, fb, policy, lo, c)
            for name, want in zip(("seq_id", "pos", "reset", "valid"), O.metadata(op, lo, c)):
                assert np.array_equal(res[name], want), name
            rag = G.Guarded(op.sum_t * fb, 0x5A)
            B.bload_unpack(plan, dense.t, fb, lo, c, rag.t)
            torch.cuda.synchronize(); rag.check()
            want = np.full(op.sum_t * fb, 0x5A, np.uint8)
            O.unpack(op, res["dense"], fb, lo, c, want)
            assert np.array_equal(rag.t.cpu().numpy(), want), (T.size, tb, fb, policy, lo, c)
