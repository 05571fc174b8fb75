"""BLoad ragged-to-block packing on B200: thin binding over libbload.so (CUDA, sm_100a).

    plan  = bload_plan(lengths_i32_cuda, t_block, seed)
    bload_pack(plan, store, frame_bytes, 0, plan.n_blocks, dense=..., seq_id=..., pos=..., reset=..., valid=...)
    bload_unpack(plan, dense_out, out_frame_bytes, 0, plan.n_blocks, ragged_out)
    bload_stats(plan.info)

The shared library is loaded on first use; nothing here computes on the CPU.
"""
from ._lib import (BloadError, Plan, PlanInfo, Sizes, bload_pack, bload_plan, bload_plan_static, bload_plan_chunks, ChunkInfo, bload_plan_async, bload_plan_finish, bload_plan_sizes, bload_rank_range,  # noqa: F401
                   bload_epoch, bload_epoch_stage_times, bload_carry_prev, bload_reset_state, bload_valid_sum, bload_var_offsets, bload_pack_var, bload_unpack_var, bload_var_offsets2d, bload_pack_var2d, bload_unpack_var2d,
                   bload_kernel_launches, bload_last_copy_kernel, bload_debug_status, bload_plan_stage_times, bload_set_plan_timing, bload_stats, bload_unpack, load, strerror)
