"""Helpers of the GPU parity tests: run the library through its C ABI, the oracle on the host,
and compare bit for bit."""
import numpy as np
import torch

import invariants
import paper_2310_10879_b200 as B
from oracle import bload_oracle as O

DEV = "cuda:0"
GUARD = 4096  # canary bytes on both sides of every output


def gpu_plan(lengths: np.ndarray, t_block: int, seed: int, check=True, policy=0):
    d_len = torch.from_numpy(np.ascontiguousarray(lengths, dtype=np.int32)).to(DEV)
    return B.bload_plan(d_len, t_block, seed, policy=policy, check=check)


def host_tables(plan) -> dict:
    return {k: v.cpu().numpy() for k, v in plan.tables().items()}


def assert_plan_equal(plan, op, maximal=None, invariants_too=True):
    """GPU plan vs oracle plan: every table and scalar, bit exact; plus the validity checker."""
    i = plan.info
    assert i.status == 0 and op.status == 0
    assert (i.n, i.t_block, i.n_blocks, i.sum_t, i.t_max) == (op.n, op.t_block, op.n_blocks, op.sum_t, op.t_max)
    assert i.first_bad_index == -1
    t = host_tables(plan)
    for name in ("offsets", "seg_seq", "seg_block", "seg_start", "block_seg_begin", "block_fill", "seq_block",
                 "seq_start"):
        a, b = t[name], getattr(op, name)
        assert a.dtype == b.dtype and a.shape == b.shape, name
        if not np.array_equal(a, b):
            bad = int(np.flatnonzero(a != b)[0])
            raise AssertionError("%s differs first at %d: gpu %s oracle %s" % (name, bad, a[bad], b[bad]))
    assert np.array_equal(t["seg_src"], op.offsets[op.seg_seq.astype(np.int64)])
    assert i.checksum == op.checksum and i.max_segs_per_block == op.max_segs_per_block
    if not invariants_too:                 # e.g. chunks with deleted frames: the "sequences" do not tile the store
        return
    if maximal is None:
        maximal = i.policy != 2            # best fit decreasing keeps several blocks open
    invariants.check_plan(op.lengths, i.t_block, i.n_blocks, t["offsets"], t["seg_seq"], t["seg_block"],
                          t["seg_start"], t["block_seg_begin"], t["block_fill"], t["seq_block"], t["seq_start"],
                          maximal=maximal)


class Guarded:
    """A device buffer with canary bytes before and after it."""

    def __init__(self, nbytes: int, fill: int = 0xEE):
        self.nbytes = nbytes
        self.raw = torch.full((nbytes + 2 * GUARD,), 0xC7, dtype=torch.uint8, device=DEV)
        self.t = self.raw[GUARD:GUARD + nbytes]
        self.t.fill_(fill)

    def check(self):
        assert bool((self.raw[:GUARD] == 0xC7).all()) and bool((self.raw[GUARD + self.nbytes:] == 0xC7).all()), \
            "write outside the output buffer"


def gpu_pack_all(plan, store_u8: torch.Tensor, fb: int, b0: int, cnt: int, pad: int, meta=True):
    tb = plan.t_block
    dense = Guarded(cnt * tb * fb)
    outs = {}
    if meta:
        outs = dict(seq_id=Guarded(cnt * tb * 4, 0x11), pos=Guarded(cnt * tb * 4, 0x11),
                    reset=Guarded(cnt * tb, 0x11), valid=Guarded(cnt * tb, 0x11))
    B.bload_pack(plan, store_u8, fb, b0, cnt, dense=dense.t,
                 seq_id=outs["seq_id"].t.view(torch.int32) if meta else None,
                 pos=outs["pos"].t.view(torch.int32) if meta else None,
                 reset=outs["reset"].t if meta else None, valid=outs["valid"].t if meta else None, pad_byte=pad)
    torch.cuda.synchronize()
    dense.check()
    for g in outs.values():
        g.check()
    res = dict(dense=dense.t.cpu().numpy().reshape(cnt, tb, fb))
    if meta:
        res.update(seq_id=outs["seq_id"].t.view(torch.int32).cpu().numpy().reshape(cnt, tb),
                   pos=outs["pos"].t.view(torch.int32).cpu().numpy().reshape(cnt, tb),
                   reset=outs["reset"].t.cpu().numpy().reshape(cnt, tb),
                   valid=outs["valid"].t.cpu().numpy().reshape(cnt, tb))
    return res, dense


def first_diff(a: np.ndarray, b: np.ndarray):
    a = a.reshape(-1); b = b.reshape(-1)
    if a.size != b.size:
        return "size %d vs %d" % (a.size, b.size)
    step = 1 << 26
    for lo in range(0, a.size, step):
        if not np.array_equal(a[lo:lo + step], b[lo:lo + step]):
            i = lo + int(np.flatnonzero(a[lo:lo + step] != b[lo:lo + step])[0])
            return "first difference at flat index %d: %s vs %s" % (i, a[i], b[i])
    return None


def full_parity(lengths: np.ndarray, t_block: int, seed: int, fb: int, out_fb: int | None = None, pad: int = 0,
                extra_blocks: int = 2, payload_seed: int = 5, policy: int = 0):
    """plan + metadata + pack + unpack of ALL blocks (plus filler blocks) against the oracle."""
    op = O.plan(lengths, t_block, seed, policy)
    plan = gpu_plan(lengths, t_block, seed, policy=policy)
    assert_plan_equal(plan, op)
    g = torch.Generator(device=DEV); g.manual_seed(payload_seed)
    store = torch.randint(0, 256, (op.sum_t * fb,), dtype=torch.uint8, device=DEV, generator=g)
    cnt = op.n_blocks + extra_blocks
    res, _ = gpu_pack_all(plan, store, fb, 0, cnt, pad)
    store_h = store.cpu().numpy()
    want = O.pack(op, store_h, fb, 0, cnt, pad)
    d = first_diff(res["dense"], want)
    assert d is None, "packed bytes: " + d
    for name, w in zip(("seq_id", "pos", "reset", "valid"), O.metadata(op, 0, cnt)):
        assert np.array_equal(res[name], w), name
    # unpack of a per-frame output of out_fb bytes per frame
    ofb = out_fb or fb
    dense_out = torch.randint(0, 256, (cnt * t_block * ofb,), dtype=torch.uint8, device=DEV, generator=g)
    rag = Guarded(op.sum_t * ofb, 0x5A)
    B.bload_unpack(plan, dense_out, ofb, 0, cnt, rag.t)
    torch.cuda.synchronize()
    rag.check()
    want_r = np.full(op.sum_t * ofb, 0x5A, np.uint8)
    O.unpack(op, dense_out.cpu().numpy(), ofb, 0, cnt, want_r)
    d = first_diff(rag.t.cpu().numpy(), want_r)
    assert d is None, "unpacked bytes: " + d
    # round trip through the GPU path alone: unpack(pack(x)) == x
    dense_dev = torch.from_numpy(res["dense"].reshape(-1)).to(DEV)
    back = Guarded(op.sum_t * fb, 0x5A)
    B.bload_unpack(plan, dense_dev, fb, 0, cnt, back.t)
    torch.cuda.synchronize()
    back.check()
    assert torch.equal(back.t, store)
    return plan, op


def expected_copy_kernels(sum_t: int, n: int, fb: int, t_block: int) -> dict:
    """Which kernel the library is documented to choose for a call (the rules stated beside launch_copy): `pack` and
    `unpack` for whole-plan calls without metadata, `unpack_range` for a block sub-range, `pack_meta` for a pack call
    that also asks for metadata and holds at most 4 Mi slots."""
    run = sum_t * fb // n
    if fb % 4 == 0 and run <= 16384:
        words = run <= 768
        if fb % 8 == 0:
            plain = dict(pack="k19_pack_walk_dense", unpack="k21_unpack_walk_ragged", unpack_range="k19_unpack_walk_dense")
        elif words:
            plain = dict(pack="k17_pack_short_runs", unpack="k18_unpack_short_runs", unpack_range="k19_unpack_walk_dense")
        else:
            plain = dict(pack="k10_pack_contig", unpack="k9_unpack_ragged",
                         unpack_range="k8_unpack_staged" if (t_block * fb) % 16 == 0 else "k7_copy<unpack>")
        plain["pack_meta"] = ("k17_pack_short_runs" if (fb % 16 == 0 or words) else "k10_pack_contig") + "<metadata>"
        return plain
    gran = fb < 4 and run <= 4096  # frames of 1 to 3 bytes in runs beyond the word-wise walks: 16-byte granules
    if fb % 4 != 0 and ((fb % 2 == 0 and run <= 1536) or run <= 384):
        up = run <= (1024 if fb % 2 == 0 else 384)
        return dict(pack="k19_pack_walk_dense",
                    unpack="k21_unpack_walk_ragged" if up else ("k25_unpack_granules" if gran else "k7_copy<unpack>"),
                    unpack_range="k19_unpack_walk_dense" if up else "k7_copy<unpack>", pack_meta="k19_pack_walk_dense")
    if gran:  # (whole-plan unpack; block sub-ranges stay on the register path)
        return dict(pack="k24_pack_granules", unpack="k25_unpack_granules", unpack_range="k7_copy<unpack>", pack_meta="k24_pack_granules")
    return dict(pack="k7_copy<pack>", unpack="k7_copy<unpack>", unpack_range="k7_copy<unpack>", pack_meta="k7_copy<pack>")
