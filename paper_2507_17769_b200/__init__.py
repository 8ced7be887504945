"""Mixed-batch paged-KV attention for one serving iteration on B200 (sm_100a).

The package is a thin Python binding over ``libpolyserve_attn.so`` (C ABI in
``include/polyserve_attn.h`` and, for the scheduler-side table consumers,
``include/polyserve_sched.h``) plus :class:`PagedAttention`, a convenience
wrapper that keeps the pool, plan and workspace of one engine together.
All arithmetic runs in the CUDA kernels; there is no CPU path.
"""
from .binding import (  # noqa: F401
    PS_STATIC_WORKSPACE_BYTES, PsError, make_shape, ps_attn_plan, ps_attn_run, ps_attn_run_static, ps_grid_row, ps_kv_alloc, ps_kv_bytes, ps_kv_free, ps_kv_gather, ps_kv_gather_fp8,
    ps_kv_status, ps_kv_write, ps_last_error, ps_plan_free, ps_plan_get_info, ps_plan_get_items, ps_plan_info,
    ps_plan_get_timing, ps_plan_opts, ps_plan_set_timing, ps_plan_set_wait_limit, ps_plan_status, ps_profile_grid, ps_shape, ps_version,
)
from .sched_binding import (  # noqa: F401
    ps_admit, ps_chunk_next, ps_chunk_predict, ps_chunk_schedule, ps_peak_kv, ps_table_add_batch_term, ps_table_build, ps_table_build_overlap, ps_table_free,
    ps_table_get_overlap,
    ps_table_from_lines, ps_table_scale,
    ps_table_get_lines, ps_table_predict, ps_table_size,
)
from .session import PagedAttention  # noqa: F401
