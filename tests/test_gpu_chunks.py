"""GPU parity of the chunking planner (bload_chunk_count, bload_plan_chunks) and of the ordinary pack / unpack /
metadata / consumer calls run on its plans, through the C ABI, against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import gpu_util as G
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import _lib
from paper_2310_10879_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _plans(T, c, tail):
    T = np.ascontiguousarray(T, np.int32)
    ch = O.chunks(T, c, tail)
    plan, ci, cseq, cfirst = B.bload_plan_chunks(torch.from_numpy(T).to(G.DEV), c, tail)
    for k in ("n_chunks", "frames_kept", "frames_deleted", "pad_frames", "sum_t", "t_max"):
        assert getattr(ci, k) == getattr(ch, k), k
    assert ci.first_bad_index == -1 and ci.n == T.size
    assert np.array_equal(cseq.cpu().numpy(), ch.chunk_seq) and np.array_equal(cfirst.cpu().numpy(), ch.chunk_first)
    op = ch.as_plan()
    # every table and the digest; the validity checker too when the chunks tile the store
    G.assert_plan_equal(plan, op, maximal=False, invariants_too=tail == O.KEEP_TAIL)
    assert plan.info.policy == 3 + tail and plan.info.n_source == T.size
    st = B.bload_stats(plan.info)
    assert st["pad_packed"] == ch.pad_frames and st["frames_deleted"] == ch.frames_deleted and st["n_blocks"] == ch.n_chunks
    return ch, plan


@pytest.mark.parametrize("tail", [O.KEEP_TAIL, O.DROP_TAIL])
@pytest.mark.parametrize("name,n,c,fb", [("toy_video", None, 7, 48), ("features_fp16", None, 30, 64), ("features_fp16", 300, 1, 16),
                                          ("tokens", 20000, 512, 4), ("tokens", 3000, 100, 4), ("heavy_tail_bf16", 2000, 128, 256),
                                          ("video_dataset_shape", None, 22, 20), ("raw_frames", 40, 60, 4100)])
def test_chunk_plans_pack_unpack_metadata(name, n, c, fb, tail):
    w = W.WORKLOADS[name]
    T = W.lengths(W.scaled(w, n) if n else w)
    ch, plan = _plans(T, c, tail)
    g = torch.Generator(device=G.DEV); g.manual_seed(c)
    store = torch.randint(0, 256, (ch.sum_t * fb,), dtype=torch.uint8, device=G.DEV, generator=g)
    store_h = store.cpu().numpy()
    for b0, cnt in ((0, ch.n_chunks + 2), (ch.n_chunks // 2, min(5, ch.n_chunks))):
        res, _ = G.gpu_pack_all(plan, store, fb, b0, cnt, 0x4D)
        d = G.first_diff(res["dense"], O.chunk_pack(ch, store_h, fb, b0, cnt, 0x4D))
        assert d is None, "packed bytes: " + d
        for nm, want in zip(("seq_id", "pos", "reset", "valid"), O.chunk_metadata(ch, b0, cnt)):
            assert np.array_equal(res[nm], want), nm
        dense_out = torch.randint(0, 256, (cnt * c * fb,), dtype=torch.uint8, device=G.DEV, generator=g)
        rag = G.Guarded(ch.sum_t * fb, 0x5A)
        B.bload_unpack(plan, dense_out, fb, b0, cnt, rag.t)
        torch.cuda.synchronize(); rag.check()
        want = np.full(ch.sum_t * fb, 0x5A, np.uint8)       # deleted frames must keep this value
        O.chunk_unpack(ch, dense_out.cpu().numpy(), fb, b0, cnt, want)
        d = G.first_diff(rag.t.cpu().numpy(), want)
        assert d is None, "unpacked bytes: " + d
    # the consumer calls see chunks as samples: nothing is carried into slot 0 of a block
    nb = ch.n_chunks
    dense = torch.from_numpy(O.chunk_pack(ch, store_h, fb, 0, nb, 0).reshape(-1)).to(G.DEV)
    prev = G.Guarded(nb * c * fb)
    B.bload_carry_prev(plan, dense, fb, 0, nb, prev.t, fill_byte=0xEE)
    torch.cuda.synchronize(); prev.check()
    want = np.full((nb, c, fb), 0xEE, np.uint8)
    d3 = dense.cpu().numpy().reshape(nb, c, fb)
    for j in range(nb):
        want[j, 1:ch.chunk_len[j]] = d3[j, :ch.chunk_len[j] - 1]
    assert np.array_equal(prev.t.cpu().numpy().reshape(nb, c, fb), want)


def test_chunk_calls_report_errors():
    T = np.array([5, 9, 0, 3], np.int32)
    _, ci, _, _ = B.bload_plan_chunks(torch.from_numpy(T).to(G.DEV), 4, check=False)
    assert ci.status == _lib.ERR_LENGTH and ci.first_bad_index == 2
    with pytest.raises(B.BloadError) as e:                    # every sequence shorter than a chunk, tails dropped
        B.bload_plan_chunks(torch.ones(10, dtype=torch.int32, device=G.DEV), 5, O.DROP_TAIL)
    assert e.value.code == _lib.ERR_ARG
    L = B.load()
    d_len = torch.full((100,), 7, dtype=torch.int32, device=G.DEV)
    work = torch.empty(int(L.bload_chunk_work_bytes(100)), dtype=torch.uint8, device=G.DEV)
    info = B.PlanInfo()
    sizes = B.bload_plan_sizes(200, 4)
    buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=G.DEV)
    import ctypes as C
    args = lambda m, wb=work.numel(), pb=buf.numel(), tail=0, c=4: (d_len.data_ptr(), 100, c, tail, m, buf.data_ptr(), pb,
                                                                    work.data_ptr(), wb, None, None, None, C.byref(info))
    assert L.bload_plan_chunks(*args(150)) == _lib.ERR_ARG            # 100 sequences of 7 frames give 200 chunks of 4
    assert L.bload_plan_chunks(*args(200)) == 0 and info.n_blocks == 200
    assert L.bload_plan_chunks(*args(200, wb=64)) == _lib.ERR_WORKSPACE
    assert L.bload_plan_chunks(*args(200, pb=1024)) == _lib.ERR_WORKSPACE
    assert L.bload_plan_chunks(*args(200, tail=2)) == _lib.ERR_ARG
    assert L.bload_plan_chunks(*args(200, c=0)) == _lib.ERR_ARG
    # per-sequence frame sizes make no sense for chunks
    plan = B.Plan(buf, info, sizes)
    L.bload_plan_chunks(*args(200))
    z = torch.zeros(4096, dtype=torch.uint8, device=G.DEV)
    with pytest.raises(B.BloadError) as e:
        B.bload_pack_var(plan, z, z.view(torch.int32), z.view(torch.int64), 16, 0, 1, z)
    assert e.value.code == _lib.ERR_UNSUPPORTED
