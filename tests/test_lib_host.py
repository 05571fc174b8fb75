"""Host-side checks of libbload that need no GPU: the library loads, exports every symbol the
header declares, and its host-only entry points behave (sizes, statistics, argument errors)."""
import ctypes as C
import os
import re

import numpy as np

import paper_2310_10879_b200 as B
from oracle import bload_oracle as O
from paper_2310_10879_b200 import _lib

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = []
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            names += re.findall(r"BLOAD_API\s+[\w\s\*]+?\b(bload_\w+)\s*\(", text)
    return names


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 9 and set(_lib.EXPORTS) <= set(names)
    L = B.load()
    for n in names:
        assert hasattr(L, n), n
    assert L.bload_version() >= 1
    assert B.strerror(0) == "ok" and "length" in B.strerror(_lib.ERR_LENGTH)


def test_bounds_checking_build_compiles_and_exports_the_same_symbols():
    from paper_2310_10879_b200 import build
    L = C.CDLL(build.build(debug=True))
    for n in _declared():
        assert hasattr(L, n), n


def test_plan_sizes_layout():
    for n, tb in [(1, 1), (8, 6), (1000, 1000), (1_000_000, 4096), (20_000, 10_000)]:
        s = B.bload_plan_sizes(n, tb)
        offs = [s.off_offsets, s.off_seg_seq, s.off_seg_block, s.off_seg_start, s.off_seg_src,
                s.off_block_seg_begin, s.off_block_fill, s.off_seq_block, s.off_seq_start, s.plan_bytes]
        need = [8 * (n + 1), 4 * n, 4 * n, 4 * n, 8 * n, 4 * (n + 1), 4 * n, 4 * n, 4 * n]
        assert offs[0] >= 256 and all(o % 256 == 0 for o in offs)
        assert all(offs[i + 1] - offs[i] >= need[i] for i in range(9))
        assert s.max_blocks == n and s.work_bytes >= 44 * n
    L = B.load()
    s = _lib.Sizes()
    assert L.bload_plan_sizes(0, 4, C.byref(s)) == _lib.ERR_ARG
    assert L.bload_plan_sizes(2**31, 4, C.byref(s)) == _lib.ERR_ARG
    assert L.bload_plan_sizes(4, 0, C.byref(s)) == _lib.ERR_ARG
    assert L.bload_plan_sizes(4, _lib.MAX_T_BLOCK + 1, C.byref(s)) == _lib.ERR_UNSUPPORTED
    assert L.bload_plan_sizes(4, 4, None) == _lib.ERR_NULL


def test_stats_match_the_oracle_and_the_paper_table():
    rng = np.random.default_rng(0)
    cases = [(7464, 166785, 94, 94, 1775)]
    for _ in range(100):
        n = int(rng.integers(1, 10**6)); tb = int(rng.integers(1, 30000)); tm = int(rng.integers(1, tb + 1))
        s = int(rng.integers(n, n * tm + 1)); nb = int(rng.integers(-(-s // tb), n + 1))
        cases.append((n, s, tm, tb, nb))
    for n, s, tm, tb, nb in cases:
        info = B.PlanInfo(status=0, t_block=tb, n=n, n_blocks=nb, sum_t=s, t_max=tm, max_segs_per_block=3)
        got = B.bload_stats(info)
        want = O.stats(n, s, tm, tb, nb)
        for k, v in want.items():
            assert got[k] == v, k
    assert B.bload_stats(B.PlanInfo(status=0, t_block=94, n=7464, n_blocks=1775, sum_t=166785, t_max=94))[
        "pad_naive_tmax"] == 534831
    L = B.load()
    st = _lib.Stats()
    assert L.bload_stats(None, C.byref(st)) == _lib.ERR_NULL
    assert L.bload_stats(C.byref(B.PlanInfo(status=-3, n=1, t_block=1, n_blocks=1, sum_t=1)), C.byref(st)) == _lib.ERR_PLAN


def test_null_and_range_errors_without_a_device():
    L = B.load()
    info = B.PlanInfo()
    assert L.bload_plan(None, 5, 4, 0, 0, None, 0, None, 0, None, C.byref(info)) == _lib.ERR_NULL
    assert info.status == _lib.ERR_NULL and info.first_bad_index == -1
    assert L.bload_plan(None, 5, 4, 0, 0, None, 0, None, 0, None, None) == _lib.ERR_NULL
    ok = B.PlanInfo(status=0, t_block=4, n=5, n_blocks=2, sum_t=7, t_max=3)
    assert L.bload_pack(None, C.byref(ok), None, 1, 0, 1, None, None, None, None, None, 0, None) == _lib.ERR_NULL
    assert L.bload_unpack(None, C.byref(ok), None, 1, 0, 1, None, None) == _lib.ERR_NULL
    assert L.bload_pack(256, None, None, 1, 0, 1, None, None, None, None, None, 0, None) == _lib.ERR_NULL
    assert L.bload_pack(256, C.byref(B.PlanInfo(status=-3)), None, 1, 0, 1, None, None, None, None, None, 0,
                        None) == _lib.ERR_PLAN
    assert L.bload_pack(256, C.byref(ok), None, 0, 0, 1, None, None, None, None, None, 0, None) == _lib.ERR_ARG
    assert L.bload_pack(264, C.byref(ok), None, 1, 0, 1, None, None, None, None, None, 0, None) == _lib.ERR_ALIGN
    out = (C.c_float * 4)()
    assert L.bload_plan_stage_times(C.byref(out)) == _lib.ERR_PLAN


def test_newer_entry_points_reject_bad_arguments_before_any_launch():
    """Errors the host can see return before the library touches the device, so they can be checked without one."""
    L = B.load()
    E = _lib
    ok = B.PlanInfo(status=0, t_block=4, n=5, n_blocks=2, sum_t=7, t_max=3)
    p = C.byref(ok)
    # consumer side
    assert L.bload_carry_prev(None, p, 256, 4, 0, 1, 512, 0, None) == E.ERR_NULL
    assert L.bload_carry_prev(256, p, None, 4, 0, 1, 512, 0, None) == E.ERR_NULL
    assert L.bload_carry_prev(256, p, 512, 4, 0, 1, 512, 0, None) == E.ERR_ARG       # in place
    assert L.bload_carry_prev(256, p, 512, 0, 0, 1, 1024, 0, None) == E.ERR_ARG      # frame size
    assert L.bload_carry_prev(256, p, 520, 4, 0, 1, 1024, 0, None) == E.ERR_ALIGN
    assert L.bload_reset_state(256, p, 0, 1, 4, 512, 16, None, None) == E.ERR_ARG    # slot == t_block
    assert L.bload_reset_state(256, p, 0, 1, 0, None, 16, None, None) == E.ERR_NULL
    assert L.bload_reset_state(256, p, 0, 1, 0, 512, 16, 8, None) == E.ERR_ALIGN     # init not 16-byte aligned
    assert L.bload_valid_sum(256, p, None, 0, 1, 512, None, None) == E.ERR_NULL
    assert L.bload_valid_sum(256, p, 512, 0, -1, 512, None, None) == E.ERR_ARG
    assert L.bload_valid_sum(256, p, 512, 0, 1, 516, None, None) == E.ERR_ALIGN
    # per-sample frame sizes
    vi = E.VarInfo()
    assert L.bload_var_offsets(None, 512, 5, 1024, None, C.byref(vi)) == E.ERR_NULL
    assert L.bload_var_offsets(256, 512, 0, 1024, None, C.byref(vi)) == E.ERR_ARG
    assert L.bload_var_offsets(256, 512, 5, 1028, None, C.byref(vi)) == E.ERR_ALIGN
    assert L.bload_var_offsets(256, 512, 5, 1024, None, None) == E.ERR_NULL
    assert L.bload_pack_var(256, p, 512, None, 1024, 16, 0, 1, 2048, 0, None) == E.ERR_NULL
    assert L.bload_pack_var(256, p, 512, 768, 1024, 0, 0, 1, 2048, 0, None) == E.ERR_ARG
    assert L.bload_unpack_var(256, p, 520, 768, 1024, 16, 0, 1, 2048, None) == E.ERR_ALIGN
    assert L.bload_pack_var2d(256, p, 512, None, 768, 1024, 2, 16, 0, 1, 2048, 0, None) == E.ERR_NULL  # rows missing
    assert L.bload_pack_var2d(256, p, 512, 640, 768, 1024, 0, 16, 0, 1, 2048, 0, None) == E.ERR_ARG    # rows_max
    # the whole step in one call
    io = E.EpochIO(512, 4, 1024, None, None, None, None, None, 0, None, 8, 0, 0)
    info = B.PlanInfo()
    assert L.bload_epoch(None, 5, 4, 0, 256, 1 << 20, 512, 1 << 20, C.byref(io), None, None, C.byref(info)) == E.ERR_NULL
    assert L.bload_epoch(256, 5, 4, 0, 256, 1 << 20, 512, 1 << 20, None, None, None, C.byref(info)) == E.ERR_NULL
    assert L.bload_epoch(256, 0, 4, 0, 256, 1 << 20, 512, 1 << 20, C.byref(io), None, None, C.byref(info)) == E.ERR_ARG
    assert L.bload_epoch(256, 5, 4, 0, 256, 16, 512, 1 << 20, C.byref(io), None, None, C.byref(info)) == E.ERR_WORKSPACE
    bad = E.EpochIO(None, 4, 1024, None, None, None, None, None, 0, None, 8, 0, 0)          # dense without a store
    assert L.bload_epoch(256, 5, 4, 0, 256, 1 << 20, 512, 1 << 20, C.byref(bad), None, None, C.byref(info)) == E.ERR_NULL
    bad = E.EpochIO(512, 4, 1024, None, None, None, None, None, 0, None, 0, 0, 0)           # no rows for the outputs
    assert L.bload_epoch(256, 5, 4, 0, 256, 1 << 20, 512, 1 << 20, C.byref(bad), None, None, C.byref(info)) == E.ERR_ARG
    bad = E.EpochIO(512, 4, 1024, None, None, None, None, None, 0, None, 8, 0, 33)          # too many chunks
    assert L.bload_epoch(256, 5, 4, 0, 256, 1 << 20, 512, 1 << 20, C.byref(bad), None, None, C.byref(info)) == E.ERR_ARG
    out5 = (C.c_float * 5)()
    assert L.bload_epoch_stage_times(C.byref(out5)) == E.ERR_PLAN
    assert L.bload_pack_repeat_last(None, p, None, 1, 0, 1, None, None, None, None, None, 0, None) == E.ERR_NULL
