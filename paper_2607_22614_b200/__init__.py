"""B200-native (sm_100a) per-GPU role-switch state transform: thin Python binding over the C ABI.

The functions here have the names and arguments of ``include/dynaresize.h`` and only marshal
arguments; every step of the path (planning, gather/cast, inverse map, chunked staging) runs inside
``libdynaresize.so``.  There is no fallback: importing the binding without the built library, or
calling a compute entry point without a CUDA device, raises.
"""
from .binding import (  # noqa: F401
    DR_BF16, DR_F32, DR_FP8_E4M3_B128, DR_OK, DrError, Plan, dr_last_error, dr_plan_create, dr_plan_create_host, dr_plan_window_host, dr_plan_destroy,
    dr_plan_query, dr_plan_segment, dr_plan_tensor, dr_reshard, dr_reshard_inverse, dr_reshard_static, dr_plan_group, dr_reshard_groups, dr_group_desc, dr_reshard_stream, dr_shard_range, stream_desc, dr_stream_desc, dr_stream_stats, dr_ctl_create, dr_ctl_observe, dr_ctl_break_even, dr_ctl_destroy, dr_stage_in, dr_stage_out, dr_stage_begin, dr_stage_wait_buffer, dr_stage_poll, dr_stage_end, StageJob, DR_STAGE_DIR_OUT, DR_STAGE_DIR_IN, dr_probe_stream, dr_host_copy, dr_diag_bulk_wait_failures, dr_diag_bulk_starve, dr_plan_ranges, dr_reshard_push, dr_range,
    dr_strerror, lib, lib_path, model_spec, src_layout, dst_layout, stage_desc,
    dr_model_spec, dr_src_layout, dr_dst_layout, dr_plan_info, dr_tensor_desc, dr_segment_desc, dr_stage_desc,
    dr_stage_stats, dr_chunk_fn, DR_MAX_STAGE_BUFS, EXPORTS,
)
