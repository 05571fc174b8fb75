"""ctypes front end of the CPU oracle (``bload_oracle.c``).

TEST INFRASTRUCTURE.  Only the tests, the smoke check and the benchmark's CPU
baseline may import this module; the GPU library never does, and this module
never imports the GPU package.  All arrays are numpy arrays in host memory.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bload_oracle.c")
_SO = os.path.join(_HERE, "libbload_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-shared", "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _SO)
    return _SO


class _PlanStruct(C.Structure):
    _fields_ = [
        ("lengths", C.c_void_p), ("n", C.c_int64), ("t_block", C.c_int32), ("seed", C.c_uint64),
        ("policy", C.c_uint32),
        ("offsets", C.c_void_p), ("seg_seq", C.c_void_p), ("seg_block", C.c_void_p), ("seg_start", C.c_void_p),
        ("block_seg_begin", C.c_void_p), ("block_fill", C.c_void_p), ("seq_block", C.c_void_p),
        ("seq_start", C.c_void_p),
        ("n_blocks", C.c_int64), ("sum_t", C.c_int64), ("t_max", C.c_int64), ("first_bad", C.c_int64),
        ("checksum", C.c_uint64), ("max_segs_per_block", C.c_int64),
    ]


class _TablesStruct(C.Structure):
    _fields_ = [
        ("n", C.c_int64), ("n_blocks", C.c_int64), ("t_block", C.c_int32),
        ("offsets", C.c_void_p), ("seg_seq", C.c_void_p), ("seg_start", C.c_void_p),
        ("block_seg_begin", C.c_void_p),
    ]


class _StatsStruct(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("n", "sum_t", "t_max", "t_block", "n_blocks", "pad_packed",
                                          "pad_naive_tmax", "pad_naive_tblock", "min_blocks")] + \
               [(k, C.c_double) for k in ("frac_packed", "frac_naive_tmax", "frac_naive_tblock",
                                          "reduction_vs_tmax", "mean_segs_per_block")]


class _ChunksStruct(C.Structure):
    _fields_ = [("lengths", C.c_void_p), ("n", C.c_int64), ("t_chunk", C.c_int32), ("tail", C.c_uint32),
                ("capacity", C.c_int64), ("chunk_seq", C.c_void_p), ("chunk_first", C.c_void_p), ("chunk_len", C.c_void_p),
                ("n_chunks", C.c_int64), ("frames_kept", C.c_int64), ("frames_deleted", C.c_int64),
                ("pad_frames", C.c_int64), ("sum_t", C.c_int64), ("t_max", C.c_int64), ("first_bad", C.c_int64)]


class _ChunkTablesStruct(C.Structure):
    _fields_ = [("n_chunks", C.c_int64), ("t_chunk", C.c_int32), ("offsets", C.c_void_p), ("chunk_seq", C.c_void_p),
                ("chunk_first", C.c_void_p), ("chunk_len", C.c_void_p)]


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_SO)
        L.oracle_philox4x64_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_philox4x64_10.restype = None
        L.oracle_seq_key.argtypes = [C.c_uint64, C.c_int64]
        L.oracle_seq_key.restype = C.c_uint32
        L.oracle_draw_word.argtypes = [C.c_uint64, C.c_int64]
        L.oracle_draw_word.restype = C.c_uint64
        L.oracle_pick.argtypes = [C.c_uint64, C.c_uint64]
        L.oracle_pick.restype = C.c_uint64
        L.oracle_offsets.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
        L.oracle_offsets.restype = None
        L.oracle_plan.argtypes = [C.POINTER(_PlanStruct)]
        L.oracle_plan.restype = C.c_int
        L.oracle_metadata.argtypes = [C.POINTER(_TablesStruct), C.c_int64, C.c_int64] + [C.c_void_p] * 4
        L.oracle_metadata.restype = C.c_int
        L.oracle_pack.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                  C.c_void_p, C.c_uint8]
        L.oracle_pack.restype = C.c_int
        L.oracle_pack_repeat_last.argtypes = L.oracle_pack.argtypes
        L.oracle_pack_repeat_last.restype = C.c_int
        L.oracle_unpack.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                    C.c_void_p]
        L.oracle_unpack.restype = C.c_int
        L.oracle_byte_offsets.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.oracle_byte_offsets.restype = None
        L.oracle_pack_var.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                      C.c_int64, C.c_int64, C.c_void_p, C.c_uint8]
        L.oracle_pack_var.restype = C.c_int
        L.oracle_unpack_var.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                        C.c_int64, C.c_int64, C.c_void_p]
        L.oracle_unpack_var.restype = C.c_int
        L.oracle_byte_offsets2d.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.oracle_byte_offsets2d.restype = None
        L.oracle_pack_var2d.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_uint8]
        L.oracle_pack_var2d.restype = C.c_int
        L.oracle_unpack_var2d.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_int64, C.c_int64, C.c_int64, C.c_int64, C.c_void_p]
        L.oracle_unpack_var2d.restype = C.c_int
        L.oracle_carry_prev.argtypes = [C.POINTER(_TablesStruct), C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                        C.c_void_p, C.c_uint8]
        L.oracle_carry_prev.restype = C.c_int
        L.oracle_reset_state.argtypes = [C.POINTER(_TablesStruct), C.c_int64, C.c_int64, C.c_int32, C.c_void_p,
                                         C.c_int64, C.c_void_p]
        L.oracle_reset_state.restype = C.c_int
        L.oracle_valid_sum.argtypes = [C.POINTER(_TablesStruct), C.c_int64, C.c_int64, C.c_void_p,
                                       C.POINTER(C.c_double), C.POINTER(C.c_int64)]
        L.oracle_valid_sum.restype = C.c_int
        L.oracle_digest.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64]
        L.oracle_digest.restype = C.c_uint64
        L.oracle_chunks.argtypes = [C.POINTER(_ChunksStruct)]
        L.oracle_chunks.restype = C.c_int
        L.oracle_chunk_metadata.argtypes = [C.POINTER(_ChunkTablesStruct), C.c_int64, C.c_int64] + [C.c_void_p] * 4
        L.oracle_chunk_metadata.restype = C.c_int
        L.oracle_chunk_pack.argtypes = [C.POINTER(_ChunkTablesStruct), C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                        C.c_void_p, C.c_uint8]
        L.oracle_chunk_pack.restype = C.c_int
        L.oracle_chunk_unpack.argtypes = [C.POINTER(_ChunkTablesStruct), C.c_void_p, C.c_int64, C.c_int64, C.c_int64,
                                          C.c_void_p]
        L.oracle_chunk_unpack.restype = C.c_int
        L.oracle_stats.argtypes = [C.POINTER(_StatsStruct)]
        L.oracle_stats.restype = C.c_int
        _lib = L
    return _lib


def _p(a: np.ndarray) -> int:
    return a.ctypes.data


def philox4x64_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint64).copy()
    k = np.asarray(key, dtype=np.uint64).copy()
    o = np.zeros(4, dtype=np.uint64)
    lib().oracle_philox4x64_10(_p(c), _p(k), _p(o))
    return o


def seq_key(seed: int, i: int) -> int:
    return int(lib().oracle_seq_key(seed, i))


def draw_word(seed: int, k: int) -> int:
    return int(lib().oracle_draw_word(seed, k))


def pick(u: int, m: int) -> int:
    return int(lib().oracle_pick(u, m))


def offsets(lengths: np.ndarray) -> np.ndarray:
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    out = np.zeros(lengths.size + 1, dtype=np.int64)
    lib().oracle_offsets(_p(lengths), lengths.size, _p(out))
    return out


@dataclass
class OraclePlan:
    status: int
    n: int
    t_block: int
    seed: int
    n_blocks: int
    sum_t: int
    t_max: int
    first_bad: int
    checksum: int
    max_segs_per_block: int
    lengths: np.ndarray
    offsets: np.ndarray
    seg_seq: np.ndarray
    seg_block: np.ndarray
    seg_start: np.ndarray
    block_seg_begin: np.ndarray
    block_fill: np.ndarray
    seq_block: np.ndarray
    seq_start: np.ndarray

    def _tables(self) -> _TablesStruct:
        return _TablesStruct(self.n, self.n_blocks, self.t_block, _p(self.offsets), _p(self.seg_seq),
                             _p(self.seg_start), _p(self.block_seg_begin))


def plan(lengths: np.ndarray, t_block: int, seed: int, policy: int = 0) -> OraclePlan:
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    n = int(lengths.size)
    m = max(n, 1)
    a = dict(offsets=np.zeros(m + 1, np.int64), seg_seq=np.zeros(m, np.int32), seg_block=np.zeros(m, np.int32),
             seg_start=np.zeros(m, np.int32), block_seg_begin=np.zeros(m + 1, np.int32),
             block_fill=np.zeros(m, np.int32), seq_block=np.zeros(m, np.int32), seq_start=np.zeros(m, np.int32))
    s = _PlanStruct(lengths=_p(lengths), n=n, t_block=t_block, seed=seed, policy=policy,
                    **{k: _p(v) for k, v in a.items()})
    rc = lib().oracle_plan(C.byref(s))
    nb = int(s.n_blocks)
    a["block_seg_begin"] = a["block_seg_begin"][: nb + 1]
    a["block_fill"] = a["block_fill"][:nb]
    return OraclePlan(status=rc, n=n, t_block=t_block, seed=seed, n_blocks=nb, sum_t=int(s.sum_t),
                      t_max=int(s.t_max), first_bad=int(s.first_bad), checksum=int(s.checksum),
                      max_segs_per_block=int(s.max_segs_per_block), lengths=lengths, **a)


def metadata(p: OraclePlan, block_begin: int, block_count: int):
    shape = (block_count, p.t_block)
    seq_id = np.empty(shape, np.int32)
    pos = np.empty(shape, np.int32)
    reset = np.empty(shape, np.uint8)
    valid = np.empty(shape, np.uint8)
    t = p._tables()
    rc = lib().oracle_metadata(C.byref(t), block_begin, block_count, _p(seq_id), _p(pos), _p(reset), _p(valid))
    assert rc == 0, rc
    return seq_id, pos, reset, valid


def pack(p: OraclePlan, store: np.ndarray, frame_bytes: int, block_begin: int, block_count: int,
         pad_byte: int = 0) -> np.ndarray:
    """store: uint8 view of the flat ragged frame store, sum_t * frame_bytes bytes."""
    store = np.ascontiguousarray(store).view(np.uint8).reshape(-1)
    assert store.size == p.sum_t * frame_bytes
    dense = np.empty((block_count, p.t_block, frame_bytes), np.uint8)
    t = p._tables()
    rc = lib().oracle_pack(C.byref(t), _p(store), frame_bytes, block_begin, block_count, _p(dense), pad_byte)
    assert rc == 0, rc
    return dense


def pack_repeat_last(p: OraclePlan, store: np.ndarray, frame_bytes: int, block_begin: int, block_count: int,
                     pad_byte: int = 0) -> np.ndarray:
    """pack(), but the padding slots of a block repeat its last frame (filler blocks: pad_byte)."""
    store = np.ascontiguousarray(store).view(np.uint8).reshape(-1)
    assert store.size == p.sum_t * frame_bytes
    dense = np.empty((block_count, p.t_block, frame_bytes), np.uint8)
    t = p._tables()
    rc = lib().oracle_pack_repeat_last(C.byref(t), _p(store), frame_bytes, block_begin, block_count, _p(dense),
                                       pad_byte)
    assert rc == 0, rc
    return dense


def unpack(p: OraclePlan, dense_out: np.ndarray, frame_bytes: int, block_begin: int, block_count: int,
           ragged_out: np.ndarray) -> np.ndarray:
    """Scatter valid slots of dense_out (blocks block_begin..) into ragged_out (uint8, in place)."""
    dense_out = np.ascontiguousarray(dense_out).view(np.uint8).reshape(-1)
    assert dense_out.size == block_count * p.t_block * frame_bytes
    assert ragged_out.dtype == np.uint8 and ragged_out.flags.c_contiguous
    assert ragged_out.size == p.sum_t * frame_bytes
    t = p._tables()
    rc = lib().oracle_unpack(C.byref(t), _p(dense_out), frame_bytes, block_begin, block_count, _p(ragged_out))
    assert rc == 0, rc
    return ragged_out


def byte_offsets(lengths: np.ndarray, frame_bytes: np.ndarray) -> np.ndarray:
    """int64[n+1]: first byte of sequence i in a store whose sequence i holds T_i frames of frame_bytes[i] bytes."""
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    frame_bytes = np.ascontiguousarray(frame_bytes, dtype=np.int32)
    assert lengths.size == frame_bytes.size
    out = np.zeros(lengths.size + 1, dtype=np.int64)
    lib().oracle_byte_offsets(_p(lengths), _p(frame_bytes), lengths.size, _p(out))
    return out


def pack_var(p: OraclePlan, store: np.ndarray, frame_bytes: np.ndarray, slot_bytes: int, block_begin: int,
             block_count: int, pad_byte: int = 0) -> np.ndarray:
    """pack() for per-sequence frame sizes: every slot has slot_bytes bytes, a smaller frame is followed by padding."""
    frame_bytes = np.ascontiguousarray(frame_bytes, dtype=np.int32)
    boff = byte_offsets(p.lengths, frame_bytes)
    store = np.ascontiguousarray(store).view(np.uint8).reshape(-1)
    assert store.size == int(boff[-1])
    dense = np.empty((block_count, p.t_block, slot_bytes), np.uint8)
    t = p._tables()
    rc = lib().oracle_pack_var(C.byref(t), _p(store), _p(frame_bytes), _p(boff), slot_bytes, block_begin, block_count,
                               _p(dense), pad_byte)
    assert rc == 0, rc
    return dense


def unpack_var(p: OraclePlan, dense_out: np.ndarray, frame_bytes: np.ndarray, slot_bytes: int, block_begin: int,
               block_count: int, ragged_out: np.ndarray) -> np.ndarray:
    frame_bytes = np.ascontiguousarray(frame_bytes, dtype=np.int32)
    boff = byte_offsets(p.lengths, frame_bytes)
    dense_out = np.ascontiguousarray(dense_out).view(np.uint8).reshape(-1)
    assert dense_out.size == block_count * p.t_block * slot_bytes
    assert ragged_out.dtype == np.uint8 and ragged_out.flags.c_contiguous and ragged_out.size == int(boff[-1])
    t = p._tables()
    rc = lib().oracle_unpack_var(C.byref(t), _p(dense_out), _p(frame_bytes), _p(boff), slot_bytes, block_begin,
                                 block_count, _p(ragged_out))
    assert rc == 0, rc
    return ragged_out


def byte_offsets2d(lengths: np.ndarray, rows: np.ndarray, row_bytes: np.ndarray) -> np.ndarray:
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    row_bytes = np.ascontiguousarray(row_bytes, dtype=np.int32)
    out = np.zeros(lengths.size + 1, dtype=np.int64)
    lib().oracle_byte_offsets2d(_p(lengths), _p(rows), _p(row_bytes), lengths.size, _p(out))
    return out


def pack_var2d(p: OraclePlan, store: np.ndarray, rows: np.ndarray, row_bytes: np.ndarray, rows_max: int,
               row_stride: int, block_begin: int, block_count: int, pad_byte: int = 0) -> np.ndarray:
    """Images of rows[i] x row_bytes[i] bytes in the top left corner of canvases of rows_max x row_stride bytes."""
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    row_bytes = np.ascontiguousarray(row_bytes, dtype=np.int32)
    boff = byte_offsets2d(p.lengths, rows, row_bytes)
    store = np.ascontiguousarray(store).view(np.uint8).reshape(-1)
    assert store.size == int(boff[-1])
    dense = np.empty((block_count, p.t_block, rows_max, row_stride), np.uint8)
    t = p._tables()
    rc = lib().oracle_pack_var2d(C.byref(t), _p(store), _p(rows), _p(row_bytes), _p(boff), rows_max, row_stride,
                                 block_begin, block_count, _p(dense), pad_byte)
    assert rc == 0, rc
    return dense


def unpack_var2d(p: OraclePlan, dense_out: np.ndarray, rows: np.ndarray, row_bytes: np.ndarray, rows_max: int,
                 row_stride: int, block_begin: int, block_count: int, ragged_out: np.ndarray) -> np.ndarray:
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    row_bytes = np.ascontiguousarray(row_bytes, dtype=np.int32)
    boff = byte_offsets2d(p.lengths, rows, row_bytes)
    dense_out = np.ascontiguousarray(dense_out).view(np.uint8).reshape(-1)
    assert dense_out.size == block_count * p.t_block * rows_max * row_stride
    assert ragged_out.dtype == np.uint8 and ragged_out.flags.c_contiguous and ragged_out.size == int(boff[-1])
    t = p._tables()
    rc = lib().oracle_unpack_var2d(C.byref(t), _p(dense_out), _p(rows), _p(row_bytes), _p(boff), rows_max, row_stride,
                                   block_begin, block_count, _p(ragged_out))
    assert rc == 0, rc
    return ragged_out


def carry_prev(p: OraclePlan, dense: np.ndarray, frame_bytes: int, block_begin: int, block_count: int,
               fill_byte: int = 0) -> np.ndarray:
    """What every slot receives from the slot before it: the previous frame of the same sequence, or fill."""
    dense = np.ascontiguousarray(dense).view(np.uint8).reshape(-1)
    assert dense.size == block_count * p.t_block * frame_bytes
    prev = np.empty((block_count, p.t_block, frame_bytes), np.uint8)
    t = p._tables()
    rc = lib().oracle_carry_prev(C.byref(t), _p(dense), frame_bytes, block_begin, block_count, _p(prev), fill_byte)
    assert rc == 0, rc
    return prev


def reset_state(p: OraclePlan, block_begin: int, block_count: int, slot: int, state: np.ndarray,
                init: np.ndarray | None = None) -> np.ndarray:
    """In place: rows of `state` ([block_count, state_bytes] uint8) whose block starts a sequence, or has no frame,
    at `slot` are replaced by `init` (zeros when None)."""
    assert state.dtype == np.uint8 and state.flags.c_contiguous and state.shape[0] == block_count
    sb = state.size // max(block_count, 1)
    if init is not None:
        init = np.ascontiguousarray(init).view(np.uint8).reshape(-1)
        assert init.size == sb
    t = p._tables()
    rc = lib().oracle_reset_state(C.byref(t), block_begin, block_count, slot, _p(state), sb,
                                  _p(init) if init is not None else None)
    assert rc == 0, rc
    return state


def valid_sum(p: OraclePlan, block_begin: int, block_count: int, values: np.ndarray) -> tuple[float, int]:
    """(sum in double precision, number) of the float32 per-slot values that sit on frames."""
    values = np.ascontiguousarray(values, dtype=np.float32).reshape(-1)
    assert values.size == block_count * p.t_block
    s, c = C.c_double(), C.c_int64()
    t = p._tables()
    rc = lib().oracle_valid_sum(C.byref(t), block_begin, block_count, _p(values), C.byref(s), C.byref(c))
    assert rc == 0, rc
    return float(s.value), int(c.value)


def stats(n: int, sum_t: int, t_max: int, t_block: int, n_blocks: int) -> dict:
    s = _StatsStruct(n=n, sum_t=sum_t, t_max=t_max, t_block=t_block, n_blocks=n_blocks)
    rc = lib().oracle_stats(C.byref(s))
    assert rc == 0, rc
    return {k: getattr(s, k) for k, _ in _StatsStruct._fields_}


# ---- the chunking strategy (a comparison system of the paper): every chunk of t_chunk frames is a sample and a block ----

KEEP_TAIL, DROP_TAIL = 0, 1


@dataclass
class OracleChunks:
    status: int
    n: int                 # sequences the chunks were cut from
    t_chunk: int
    tail: int
    n_chunks: int
    frames_kept: int
    frames_deleted: int
    pad_frames: int
    sum_t: int
    t_max: int
    first_bad: int
    lengths: np.ndarray
    offsets: np.ndarray    # int64[n+1] of the original sequences
    chunk_seq: np.ndarray
    chunk_first: np.ndarray
    chunk_len: np.ndarray

    def _tables(self) -> _ChunkTablesStruct:
        return _ChunkTablesStruct(self.n_chunks, self.t_chunk, _p(self.offsets), _p(self.chunk_seq), _p(self.chunk_first),
                                  _p(self.chunk_len))

    def as_plan(self) -> OraclePlan:
        """The same chunks written as plan tables: chunk j is "sequence" j and fills block j from slot 0; its entry of
        `offsets` is its first frame in the original store ([n_chunks] = all frames of that store)."""
        m = self.n_chunks
        ar = np.arange(m, dtype=np.int32)
        zeros = np.zeros(m, np.int32)
        off = np.empty(m + 1, np.int64)
        off[:m] = self.offsets[self.chunk_seq.astype(np.int64)] + self.chunk_first
        off[m] = self.sum_t
        digest = int(lib().oracle_digest(_p(ar), _p(zeros), _p(ar), m))
        return OraclePlan(status=self.status, n=m, t_block=self.t_chunk, seed=0, n_blocks=m, sum_t=self.sum_t,
                          t_max=int(self.chunk_len.max()) if m else 0, first_bad=self.first_bad, checksum=digest,
                          max_segs_per_block=1 if m else 0,
                          lengths=self.chunk_len.copy(), offsets=off, seg_seq=ar.copy(), seg_block=ar.copy(),
                          seg_start=zeros.copy(), block_seg_begin=np.arange(m + 1, dtype=np.int32),
                          block_fill=self.chunk_len.copy(), seq_block=ar.copy(), seq_start=zeros.copy())


def chunks(lengths: np.ndarray, t_chunk: int, tail: int = KEEP_TAIL) -> OracleChunks:
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    n = int(lengths.size)
    s = _ChunksStruct(lengths=_p(lengths), n=n, t_chunk=t_chunk, tail=tail, capacity=0)
    rc = lib().oracle_chunks(C.byref(s))                      # first pass: count
    m = int(s.n_chunks) if rc == 0 else 0
    seq, first, ln = (np.zeros(max(m, 1), np.int32) for _ in range(3))
    if rc == 0:
        s = _ChunksStruct(lengths=_p(lengths), n=n, t_chunk=t_chunk, tail=tail, capacity=m, chunk_seq=_p(seq),
                          chunk_first=_p(first), chunk_len=_p(ln))
        rc = lib().oracle_chunks(C.byref(s))
    return OracleChunks(status=rc, n=n, t_chunk=t_chunk, tail=tail, n_chunks=m, frames_kept=int(s.frames_kept),
                        frames_deleted=int(s.frames_deleted), pad_frames=int(s.pad_frames), sum_t=int(s.sum_t),
                        t_max=int(s.t_max), first_bad=int(s.first_bad), lengths=lengths,
                        offsets=offsets(lengths) if n else np.zeros(1, np.int64), chunk_seq=seq[:m], chunk_first=first[:m],
                        chunk_len=ln[:m])


def chunk_metadata(c: OracleChunks, block_begin: int, block_count: int):
    shape = (block_count, c.t_chunk)
    seq_id = np.empty(shape, np.int32); pos = np.empty(shape, np.int32)
    reset = np.empty(shape, np.uint8); valid = np.empty(shape, np.uint8)
    t = c._tables()
    rc = lib().oracle_chunk_metadata(C.byref(t), block_begin, block_count, _p(seq_id), _p(pos), _p(reset), _p(valid))
    assert rc == 0, rc
    return seq_id, pos, reset, valid


def chunk_pack(c: OracleChunks, store: np.ndarray, frame_bytes: int, block_begin: int, block_count: int,
               pad_byte: int = 0) -> np.ndarray:
    store = np.ascontiguousarray(store).view(np.uint8).reshape(-1)
    assert store.size == c.sum_t * frame_bytes
    dense = np.empty((block_count, c.t_chunk, frame_bytes), np.uint8)
    t = c._tables()
    rc = lib().oracle_chunk_pack(C.byref(t), _p(store), frame_bytes, block_begin, block_count, _p(dense), pad_byte)
    assert rc == 0, rc
    return dense


def chunk_unpack(c: OracleChunks, dense_out: np.ndarray, frame_bytes: int, block_begin: int, block_count: int,
                 ragged_out: np.ndarray) -> np.ndarray:
    dense_out = np.ascontiguousarray(dense_out).view(np.uint8).reshape(-1)
    assert dense_out.size == block_count * c.t_chunk * frame_bytes
    assert ragged_out.dtype == np.uint8 and ragged_out.flags.c_contiguous and ragged_out.size == c.sum_t * frame_bytes
    t = c._tables()
    rc = lib().oracle_chunk_unpack(C.byref(t), _p(dense_out), frame_bytes, block_begin, block_count, _p(ragged_out))
    assert rc == 0, rc
    return ragged_out
