"""ctypes binding of libbload.so: argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; torch is used for device memory
and streams.  There is no CPU fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("BLOAD_LIBRARY") or os.path.join(_HERE, "libbload.so")  # override: a build to compare

OK = 0
ERR_NULL, ERR_ARG, ERR_LENGTH, ERR_WORKSPACE, ERR_ALIGN = -1, -2, -3, -4, -5
ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT, ERR_PLAN = -6, -7, -8, -9
MAX_T_BLOCK = 32768

EXPORTS = ("bload_plan_sizes", "bload_plan", "bload_plan_async", "bload_plan_finish", "bload_rank_range", "bload_pack", "bload_unpack", "bload_stats", "bload_epoch", "bload_epoch_stage_times",
           "bload_pack_repeat_last", "bload_var_offsets", "bload_pack_var", "bload_unpack_var", "bload_var_offsets2d", "bload_pack_var2d",
           "bload_unpack_var2d", "bload_carry_prev", "bload_reset_state", "bload_valid_sum",
           "bload_plan_static", "bload_chunk_work_bytes", "bload_chunk_count", "bload_plan_chunks", "bload_set_plan_timing", "bload_plan_stage_times", "bload_kernel_launches", "bload_last_copy_kernel", "bload_debug_status", "bload_bulk_copy_timeouts",
           "bload_strerror", "bload_version")


class Sizes(C.Structure):
    _fields_ = [("plan_bytes", C.c_size_t), ("work_bytes", C.c_size_t), ("max_blocks", C.c_int64)] + \
               [(k, C.c_size_t) for k in ("off_offsets", "off_seg_seq", "off_seg_block", "off_seg_start",
                                          "off_seg_src", "off_block_seg_begin", "off_block_fill",
                                          "off_seq_block", "off_seq_start")]


class PlanInfo(C.Structure):
    _fields_ = [("status", C.c_int32), ("t_block", C.c_int32), ("n", C.c_int64), ("n_blocks", C.c_int64),
                ("sum_t", C.c_int64), ("t_max", C.c_int64), ("first_bad_index", C.c_int64),
                ("checksum", C.c_uint64), ("max_segs_per_block", C.c_int64), ("seed", C.c_uint64),
                ("policy", C.c_uint32), ("n_source", C.c_uint32)]


class Stats(C.Structure):
    _fields_ = [(k, C.c_int64) for k in ("n", "sum_t", "t_max", "t_block", "n_blocks", "pad_packed",
                                          "pad_naive_tmax", "pad_naive_tblock", "min_blocks")] + \
               [(k, C.c_double) for k in ("frac_packed", "frac_naive_tmax", "frac_naive_tblock",
                                          "reduction_vs_tmax", "mean_segs_per_block")] + \
               [("max_segs_per_block", C.c_int64), ("frames_deleted", C.c_int64)]


class EpochIO(C.Structure):
    _fields_ = [("d_store", C.c_void_p), ("frame_bytes", C.c_int64), ("d_dense", C.c_void_p),
                ("d_seq_id", C.c_void_p), ("d_pos", C.c_void_p), ("d_reset", C.c_void_p), ("d_valid", C.c_void_p),
                ("d_dense_out", C.c_void_p), ("out_frame_bytes", C.c_int64), ("d_ragged_out", C.c_void_p),
                ("block_capacity", C.c_int64), ("pad_byte", C.c_uint8), ("chunks", C.c_uint8), ("reserved_", C.c_uint8 * 6)]


class ChunkInfo(C.Structure):
    _fields_ = [("status", C.c_int32), ("tail", C.c_uint32), ("t_chunk", C.c_int32), ("reserved_", C.c_int32)] + \
               [(k, C.c_int64) for k in ("n", "n_chunks", "frames_kept", "frames_deleted", "pad_frames", "sum_t", "t_max",
                                          "first_bad_index")]


class VarInfo(C.Structure):
    _fields_ = [("total_bytes", C.c_int64), ("max_frame_bytes", C.c_int64), ("first_bad_index", C.c_int64),
                ("max_rows", C.c_int64)]


class BloadError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, strerror(code), code))


_lib = None


def load() -> C.CDLL:
    """Load libbload.so.  Raises if it has not been built (python -m paper_2310_10879_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if "BLOAD_LIBRARY" not in os.environ:
        # a missing or stale in-tree library is (re)built from the CUDA sources; if that is impossible, fail loudly:
        # a library built from other sources than the ones in this tree must never run unnoticed
        from . import build as _build
        try:
            _build.build()
        except Exception as exc:
            what = "is missing" if not os.path.exists(LIB_PATH) else "was built from other sources than this tree's"
            raise RuntimeError("libbload.so at %s %s and could not be rebuilt (%s); there is no CPU fallback.  Build it "
                               "with `python -m paper_2310_10879_b200.build`, or name a library to load with "
                               "BLOAD_LIBRARY" % (LIB_PATH, what, exc)) from exc
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libbload.so is missing at %s: build it with `python -m paper_2310_10879_b200.build` "
                           "(there is no CPU fallback)" % LIB_PATH)
    L = C.CDLL(LIB_PATH)
    vp, i64, i32, u64, u32, u8 = C.c_void_p, C.c_int64, C.c_int32, C.c_uint64, C.c_uint32, C.c_uint8
    L.bload_plan_sizes.argtypes = [i64, i32, C.POINTER(Sizes)]
    L.bload_plan.argtypes = [vp, i64, i32, u64, u32, vp, C.c_size_t, vp, C.c_size_t, vp, C.POINTER(PlanInfo)]
    L.bload_plan_async.argtypes = [vp, i64, i32, u64, u32, vp, C.c_size_t, vp, C.c_size_t, vp]
    L.bload_chunk_work_bytes.argtypes = [i64]
    L.bload_chunk_count.argtypes = [vp, i64, i32, u32, vp, C.c_size_t, vp, C.POINTER(ChunkInfo)]
    L.bload_plan_chunks.argtypes = [vp, i64, i32, u32, i64, vp, C.c_size_t, vp, C.c_size_t, vp, vp, vp, C.POINTER(PlanInfo)]
    L.bload_plan_static.argtypes = [vp, i64, i32, u64, u32, vp, C.c_size_t, vp, C.POINTER(PlanInfo)]
    L.bload_plan_finish.argtypes = [vp, vp, C.POINTER(PlanInfo)]
    L.bload_rank_range.argtypes = [i64, i32, i32, i32, C.POINTER(i64), C.POINTER(i64)]
    L.bload_pack.argtypes = [vp, C.POINTER(PlanInfo), vp, i64, i64, i64, vp, vp, vp, vp, vp, u8, vp]
    L.bload_pack_repeat_last.argtypes = L.bload_pack.argtypes
    L.bload_unpack.argtypes = [vp, C.POINTER(PlanInfo), vp, i64, i64, i64, vp, vp]
    L.bload_stats.argtypes = [C.POINTER(PlanInfo), C.POINTER(Stats)]
    L.bload_var_offsets.argtypes = [vp, vp, i64, vp, vp, C.POINTER(VarInfo)]
    L.bload_pack_var.argtypes = [vp, C.POINTER(PlanInfo), vp, vp, vp, i64, i64, i64, vp, u8, vp]
    L.bload_unpack_var.argtypes = [vp, C.POINTER(PlanInfo), vp, vp, vp, i64, i64, i64, vp, vp]
    L.bload_var_offsets2d.argtypes = [vp, vp, vp, i64, vp, vp, C.POINTER(VarInfo)]
    L.bload_pack_var2d.argtypes = [vp, C.POINTER(PlanInfo), vp, vp, vp, vp, i64, i64, i64, i64, vp, u8, vp]
    L.bload_unpack_var2d.argtypes = [vp, C.POINTER(PlanInfo), vp, vp, vp, vp, i64, i64, i64, i64, vp, vp]
    L.bload_carry_prev.argtypes = [vp, C.POINTER(PlanInfo), vp, i64, i64, i64, vp, u8, vp]
    L.bload_reset_state.argtypes = [vp, C.POINTER(PlanInfo), i64, i64, i32, vp, i64, vp, vp]
    L.bload_valid_sum.argtypes = [vp, C.POINTER(PlanInfo), vp, i64, i64, vp, vp, vp]
    L.bload_epoch.argtypes = [vp, i64, i32, u64, vp, C.c_size_t, vp, C.c_size_t, C.POINTER(EpochIO), vp, vp,
                              C.POINTER(PlanInfo)]
    L.bload_epoch_stage_times.argtypes = [C.POINTER(C.c_float * 5)]
    L.bload_set_plan_timing.argtypes = [C.c_int]
    L.bload_plan_stage_times.argtypes = [C.POINTER(C.c_float * 4)]
    L.bload_strerror.argtypes = [C.c_int]
    L.bload_strerror.restype = C.c_char_p
    L.bload_last_copy_kernel.argtypes = [C.c_int]
    L.bload_debug_status.argtypes = [C.POINTER(C.c_uint64 * 4), C.c_int]
    L.bload_version.argtypes = []
    L.bload_kernel_launches.argtypes = []
    for name in EXPORTS:
        if name not in ("bload_strerror", "bload_kernel_launches", "bload_last_copy_kernel", "bload_debug_status", "bload_bulk_copy_timeouts", "bload_chunk_work_bytes"):
            getattr(L, name).restype = C.c_int
    L.bload_kernel_launches.restype = C.c_int64
    L.bload_bulk_copy_timeouts.argtypes = []
    L.bload_bulk_copy_timeouts.restype = C.c_int64
    L.bload_chunk_work_bytes.restype = C.c_size_t
    L.bload_last_copy_kernel.restype = C.c_char_p
    _lib = L
    return L


def strerror(code: int) -> str:
    return load().bload_strerror(code).decode()


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int | None:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


def bload_plan_sizes(n: int, t_block: int) -> Sizes:
    s = Sizes()
    rc = load().bload_plan_sizes(n, t_block, C.byref(s))
    if rc:
        raise BloadError(rc, "bload_plan_sizes")
    return s


@dataclass
class Plan:
    """A device plan: the raw buffer, its host scalars, and typed views of its tables (device tensors
    that alias the buffer)."""
    buf: "object"
    info: PlanInfo
    sizes: Sizes

    def _view(self, off: int, count: int, dtype):
        import torch
        esz = torch.empty((), dtype=dtype).element_size()
        return self.buf[off: off + count * esz].view(dtype)

    @property
    def n(self): return int(self.info.n)
    @property
    def t_block(self): return int(self.info.t_block)
    @property
    def n_blocks(self): return int(self.info.n_blocks)
    @property
    def sum_t(self): return int(self.info.sum_t)

    def tables(self) -> dict:
        import torch
        n, nb, s = self.n, self.n_blocks, self.sizes
        return dict(
            offsets=self._view(s.off_offsets, n + 1, torch.int64),
            seg_seq=self._view(s.off_seg_seq, n, torch.int32),
            seg_block=self._view(s.off_seg_block, n, torch.int32),
            seg_start=self._view(s.off_seg_start, n, torch.int32),
            seg_src=self._view(s.off_seg_src, n, torch.int64),
            block_seg_begin=self._view(s.off_block_seg_begin, nb + 1, torch.int32),
            block_fill=self._view(s.off_block_fill, nb, torch.int32),
            seq_block=self._view(s.off_seq_block, n, torch.int32),
            seq_start=self._view(s.off_seq_start, n, torch.int32),
        )


def bload_plan(lengths, t_block: int, seed: int, policy: int = 0, stream=None, work=None, plan_buf=None,
               check: bool = True) -> Plan:
    """lengths: CUDA int32 tensor [n].  Returns a Plan whose tables live in device memory."""
    import torch
    if not lengths.is_cuda or lengths.dtype != torch.int32 or not lengths.is_contiguous():
        raise TypeError("lengths must be a contiguous CUDA int32 tensor")
    n = lengths.numel()
    sizes = bload_plan_sizes(n, t_block)
    dev = lengths.device
    if plan_buf is None:
        plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=dev)
    if work is None:
        work = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=dev)
    info = PlanInfo()
    rc = load().bload_plan(lengths.data_ptr(), n, t_block, seed, policy, plan_buf.data_ptr(), plan_buf.numel(),
                           work.data_ptr(), work.numel(), _stream(stream), C.byref(info))
    if rc and check:
        err = BloadError(rc, "bload_plan")
        err.info = info
        raise err
    return Plan(plan_buf, info, sizes)


def bload_epoch(lengths, t_block: int, seed: int, block_capacity: int, store=None, frame_bytes: int = 0, dense=None,
                seq_id=None, pos=None, reset=None, valid=None, pad_byte: int = 0, dense_out=None,
                out_frame_bytes: int = 0, ragged_out=None, stream=None, side_stream=None, work=None, plan_buf=None,
                check: bool = True, chunks: int = 0) -> Plan:
    """Plan, metadata, pack and unpack of a whole epoch in one call; the copies of finished blocks run on
    `side_stream` while the plan is still being built on `stream`.  Same results as bload_plan + bload_pack +
    bload_unpack over blocks [0, block_capacity).  All outputs are complete when the call returns."""
    import torch
    if not lengths.is_cuda or lengths.dtype != torch.int32 or not lengths.is_contiguous():
        raise TypeError("lengths must be a contiguous CUDA int32 tensor")
    n = lengths.numel()
    sizes = bload_plan_sizes(n, t_block)
    if plan_buf is None:
        plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=lengths.device)
    if work is None:
        work = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=lengths.device)
    io = EpochIO(_ptr(store), frame_bytes, _ptr(dense), _ptr(seq_id), _ptr(pos), _ptr(reset), _ptr(valid),
                 _ptr(dense_out), out_frame_bytes, _ptr(ragged_out), block_capacity, pad_byte, chunks)
    info = PlanInfo()
    side = None if side_stream is None else (side_stream.cuda_stream or None)
    rc = load().bload_epoch(lengths.data_ptr(), n, t_block, seed, plan_buf.data_ptr(), plan_buf.numel(),
                            work.data_ptr(), work.numel(), C.byref(io), _stream(stream), side, C.byref(info))
    if rc and check:
        err = BloadError(rc, "bload_epoch")
        err.info = info
        raise err
    return Plan(plan_buf, info, sizes)


def bload_epoch_stage_times() -> list[float]:
    out = (C.c_float * 5)()
    rc = load().bload_epoch_stage_times(C.byref(out))
    if rc:
        raise BloadError(rc, "bload_epoch_stage_times")
    return [float(x) for x in out]


def bload_plan_async(lengths, t_block: int, seed: int, policy: int = 0, stream=None, work=None, plan_buf=None):
    """Enqueue a plan without waiting for it.  Returns (plan_buf, work, sizes); keep all three alive and
    call bload_plan_finish(plan_buf, sizes, stream) to obtain the Plan."""
    import torch
    if not lengths.is_cuda or lengths.dtype != torch.int32 or not lengths.is_contiguous():
        raise TypeError("lengths must be a contiguous CUDA int32 tensor")
    n = lengths.numel()
    sizes = bload_plan_sizes(n, t_block)
    if plan_buf is None:
        plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=lengths.device)
    if work is None:
        work = torch.empty(sizes.work_bytes, dtype=torch.uint8, device=lengths.device)
    rc = load().bload_plan_async(lengths.data_ptr(), n, t_block, seed, policy, plan_buf.data_ptr(), plan_buf.numel(),
                                 work.data_ptr(), work.numel(), _stream(stream))
    if rc:
        raise BloadError(rc, "bload_plan_async")
    return plan_buf, work, sizes


def bload_plan_finish(plan_buf, sizes: Sizes, stream=None, check: bool = True) -> Plan:
    info = PlanInfo()
    rc = load().bload_plan_finish(plan_buf.data_ptr(), _stream(stream), C.byref(info))
    if rc and check:
        err = BloadError(rc, "bload_plan_finish")
        err.info = info
        raise err
    return Plan(plan_buf, info, sizes)


def bload_pack(plan: Plan, store, frame_bytes: int, block_begin: int, block_count: int, dense=None, seq_id=None,
               pos=None, reset=None, valid=None, pad_byte: int = 0, stream=None, repeat_last: bool = False) -> None:
    """store: CUDA tensor holding the flat ragged frames; dense/seq_id/pos/reset/valid: CUDA outputs or None.
    repeat_last: padding slots repeat the block's last frame (bload_pack_repeat_last) instead of pad_byte."""
    fn = load().bload_pack_repeat_last if repeat_last else load().bload_pack
    rc = fn(plan.buf.data_ptr(), C.byref(plan.info), _ptr(store), frame_bytes, block_begin,
                           block_count, _ptr(dense), _ptr(seq_id), _ptr(pos), _ptr(reset), _ptr(valid), pad_byte,
                           _stream(stream))
    if rc:
        raise BloadError(rc, "bload_pack")


def bload_unpack(plan: Plan, dense_out, out_frame_bytes: int, block_begin: int, block_count: int, ragged_out,
                 stream=None) -> None:
    rc = load().bload_unpack(plan.buf.data_ptr(), C.byref(plan.info), _ptr(dense_out), out_frame_bytes, block_begin,
                             block_count, _ptr(ragged_out), _stream(stream))
    if rc:
        raise BloadError(rc, "bload_unpack")


def bload_var_offsets(lengths, frame_bytes, stream=None):
    """Byte offsets of a store whose sequence i holds lengths[i] frames of frame_bytes[i] bytes (CUDA int32 tensors).
    Returns (byte_offsets int64 CUDA tensor [n+3], VarInfo); the first n+1 entries are the offsets."""
    import torch
    n = lengths.numel()
    out = torch.empty(n + 3, dtype=torch.int64, device=lengths.device)
    info = VarInfo()
    rc = load().bload_var_offsets(lengths.data_ptr(), frame_bytes.data_ptr(), n, out.data_ptr(), _stream(stream),
                                  C.byref(info))
    if rc:
        err = BloadError(rc, "bload_var_offsets")
        err.info = info
        raise err
    return out, info


def bload_pack_var(plan: Plan, store, frame_bytes, byte_offsets, slot_bytes: int, block_begin: int, block_count: int,
                   dense, pad_byte: int = 0, stream=None) -> None:
    rc = load().bload_pack_var(plan.buf.data_ptr(), C.byref(plan.info), _ptr(store), _ptr(frame_bytes),
                               _ptr(byte_offsets), slot_bytes, block_begin, block_count, _ptr(dense), pad_byte,
                               _stream(stream))
    if rc:
        raise BloadError(rc, "bload_pack_var")


def bload_unpack_var(plan: Plan, dense_out, frame_bytes, byte_offsets, slot_bytes: int, block_begin: int,
                     block_count: int, ragged_out, stream=None) -> None:
    rc = load().bload_unpack_var(plan.buf.data_ptr(), C.byref(plan.info), _ptr(dense_out), _ptr(frame_bytes),
                                 _ptr(byte_offsets), slot_bytes, block_begin, block_count, _ptr(ragged_out),
                                 _stream(stream))
    if rc:
        raise BloadError(rc, "bload_unpack_var")


def bload_var_offsets2d(lengths, rows, row_bytes, stream=None):
    """Byte offsets of a store whose sequence i holds lengths[i] images of rows[i] x row_bytes[i] bytes.
    Returns (byte_offsets int64 CUDA tensor [n+4], VarInfo)."""
    import torch
    n = lengths.numel()
    out = torch.empty(n + 4, dtype=torch.int64, device=lengths.device)
    info = VarInfo()
    rc = load().bload_var_offsets2d(lengths.data_ptr(), rows.data_ptr(), row_bytes.data_ptr(), n, out.data_ptr(),
                                    _stream(stream), C.byref(info))
    if rc:
        err = BloadError(rc, "bload_var_offsets2d")
        err.info = info
        raise err
    return out, info


def bload_pack_var2d(plan: Plan, store, rows, row_bytes, byte_offsets, rows_max: int, row_stride: int,
                     block_begin: int, block_count: int, dense, pad_byte: int = 0, stream=None) -> None:
    rc = load().bload_pack_var2d(plan.buf.data_ptr(), C.byref(plan.info), _ptr(store), _ptr(rows), _ptr(row_bytes),
                                 _ptr(byte_offsets), rows_max, row_stride, block_begin, block_count, _ptr(dense),
                                 pad_byte, _stream(stream))
    if rc:
        raise BloadError(rc, "bload_pack_var2d")


def bload_unpack_var2d(plan: Plan, dense_out, rows, row_bytes, byte_offsets, rows_max: int, row_stride: int,
                       block_begin: int, block_count: int, ragged_out, stream=None) -> None:
    rc = load().bload_unpack_var2d(plan.buf.data_ptr(), C.byref(plan.info), _ptr(dense_out), _ptr(rows),
                                   _ptr(row_bytes), _ptr(byte_offsets), rows_max, row_stride, block_begin, block_count,
                                   _ptr(ragged_out), _stream(stream))
    if rc:
        raise BloadError(rc, "bload_unpack_var2d")


def bload_carry_prev(plan: Plan, dense, frame_bytes: int, block_begin: int, block_count: int, prev,
                     fill_byte: int = 0, stream=None) -> None:
    """prev[q, s] = dense[q, s-1] where a sequence continues at slot s, fill_byte elsewhere (CUDA tensors)."""
    rc = load().bload_carry_prev(plan.buf.data_ptr(), C.byref(plan.info), _ptr(dense), frame_bytes, block_begin,
                                 block_count, _ptr(prev), fill_byte, _stream(stream))
    if rc:
        raise BloadError(rc, "bload_carry_prev")


def bload_reset_state(plan: Plan, block_begin: int, block_count: int, slot: int, state, state_bytes: int,
                      init=None, stream=None) -> None:
    """Re-initialise, in place, the rows of `state` whose block does not continue a sequence at `slot`."""
    rc = load().bload_reset_state(plan.buf.data_ptr(), C.byref(plan.info), block_begin, block_count, slot,
                                  _ptr(state), state_bytes, _ptr(init), _stream(stream))
    if rc:
        raise BloadError(rc, "bload_reset_state")


def bload_valid_sum(plan: Plan, values, block_begin: int, block_count: int, block_sum, total=None,
                    stream=None) -> None:
    """block_sum[q] (float64 CUDA tensor) = sum of the float32 values on the frames of block q; total = [sum, frames]."""
    rc = load().bload_valid_sum(plan.buf.data_ptr(), C.byref(plan.info), _ptr(values), block_begin, block_count,
                                _ptr(block_sum), _ptr(total), _stream(stream))
    if rc:
        raise BloadError(rc, "bload_valid_sum")


def bload_stats(info: PlanInfo) -> dict:
    s = Stats()
    rc = load().bload_stats(C.byref(info), C.byref(s))
    if rc:
        raise BloadError(rc, "bload_stats")
    return {k: getattr(s, k) for k, _ in Stats._fields_}


def bload_set_plan_timing(enable: bool) -> None:
    load().bload_set_plan_timing(1 if enable else 0)


def bload_plan_stage_times() -> list[float]:
    out = (C.c_float * 4)()
    rc = load().bload_plan_stage_times(C.byref(out))
    if rc:
        raise BloadError(rc, "bload_plan_stage_times")
    return [float(x) for x in out]


def bload_kernel_launches() -> int:
    return int(load().bload_kernel_launches())


def bload_debug_status(clear: bool = False):
    """[refused accesses, kernel number of the first, 0 read / 1 write, address] of the bounds-checking build
    (BLOAD_LIBRARY=.../libbload_debug.so); None from the ordinary build."""
    out = (C.c_uint64 * 4)()
    rc = load().bload_debug_status(C.byref(out), 1 if clear else 0)
    if rc == ERR_UNSUPPORTED:
        return None
    if rc:
        raise BloadError(rc, "bload_debug_status")
    return [int(x) for x in out]


KEEP_TAIL, DROP_TAIL = 0, 1


def bload_plan_chunks(lengths, t_chunk: int, tail: int = KEEP_TAIL, stream=None, check: bool = True):
    """The chunking strategy of the paper's comparison ("sampling"): every chunk of t_chunk frames of every sequence is a
    sample and a block.  Returns (Plan over the chunks, ChunkInfo, chunk_seq, chunk_first); the two int32 CUDA tensors
    name, per chunk, the sequence it was cut from and its first frame there.  Two calls into the library: the count
    (the plan cannot be sized before it), then the plan."""
    import torch
    if not lengths.is_cuda or lengths.dtype != torch.int32 or not lengths.is_contiguous():
        raise TypeError("lengths must be a contiguous CUDA int32 tensor")
    n = lengths.numel()
    L = load()
    work = torch.empty(max(int(L.bload_chunk_work_bytes(n)), 256), dtype=torch.uint8, device=lengths.device)
    ci = ChunkInfo()
    rc = L.bload_chunk_count(lengths.data_ptr(), n, t_chunk, tail, work.data_ptr(), work.numel(), _stream(stream), C.byref(ci))
    if rc:
        err = BloadError(rc, "bload_chunk_count")
        err.info = ci
        if check:
            raise err
        return None, ci, None, None
    m = int(ci.n_chunks)
    if m < 1:
        if check:
            raise BloadError(ERR_ARG, "bload_plan_chunks (no chunk is kept)")
        return None, ci, None, None
    sizes = bload_plan_sizes(m, t_chunk)
    plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=lengths.device)
    chunk_seq = torch.empty(m, dtype=torch.int32, device=lengths.device)
    chunk_first = torch.empty(m, dtype=torch.int32, device=lengths.device)
    info = PlanInfo()
    rc = L.bload_plan_chunks(lengths.data_ptr(), n, t_chunk, tail, m, plan_buf.data_ptr(), plan_buf.numel(), work.data_ptr(),
                             work.numel(), chunk_seq.data_ptr(), chunk_first.data_ptr(), _stream(stream), C.byref(info))
    if rc and check:
        err = BloadError(rc, "bload_plan_chunks")
        err.info = info
        raise err
    return Plan(plan_buf, info, sizes), ci, chunk_seq, chunk_first


COPY_CALLS = {"pack": 0, "unpack": 1, "carry_prev": 2, "pack_var": 3, "unpack_var": 4}


def bload_last_copy_kernel(which: str) -> str:
    """Name of the copy kernel the last bload_pack / unpack / carry_prev / pack_var / unpack_var call of this thread chose."""
    return load().bload_last_copy_kernel(COPY_CALLS[which]).decode()


STATIC_MAX_N = 65536


def bload_plan_static(lengths, t_block: int, seed: int, policy: int = 0, stream=None, plan_buf=None,
                      check: bool = True) -> Plan:
    """bload_plan without a caller-provided scratch buffer, for callers that cannot allocate device
    memory (for example a loader thread beside a training job whose allocator owns the device).
    The library's built-in scratch array is used instead, which caps n at STATIC_MAX_N; calls that
    overlap on the GPU race on that array.  policy: 0 or 1 (best fit decreasing, 2, does not fit the
    array and raises ERR_UNSUPPORTED).  Pass a pre-made `plan_buf` to avoid every allocation; without
    one this wrapper (not the library) allocates the plan buffer with torch."""
    import torch
    if not lengths.is_cuda or lengths.dtype != torch.int32 or not lengths.is_contiguous():
        raise TypeError("lengths must be a contiguous CUDA int32 tensor")
    fn = load().bload_plan_static
    n = lengths.numel()
    sizes = bload_plan_sizes(n, t_block)
    if plan_buf is None:
        plan_buf = torch.empty(sizes.plan_bytes, dtype=torch.uint8, device=lengths.device)
    info = PlanInfo()
    rc = fn(lengths.data_ptr(), n, t_block, seed, policy, plan_buf.data_ptr(), plan_buf.numel(), _stream(stream),
            C.byref(info))
    if rc and check:
        err = BloadError(rc, "bload_plan_static")
        err.info = info
        raise err
    return Plan(plan_buf, info, sizes)


def bload_rank_range(n_blocks: int, world_size: int, rank: int, batch_blocks: int = 1) -> tuple[int, int]:
    """(first block, number of blocks) of one data-parallel rank; the same count on every rank, rounded up to whole
    batches (blocks beyond n_blocks are packed as padding)."""
    b, c = C.c_int64(), C.c_int64()
    rc = load().bload_rank_range(n_blocks, world_size, rank, batch_blocks, C.byref(b), C.byref(c))
    if rc:
        raise BloadError(rc, "bload_rank_range")
    return int(b.value), int(c.value)
