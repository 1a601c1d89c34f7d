"""CoWindow Attention for B200: thin Python binding over the C-ABI library libcowa.so.

Every step of the operator runs in the library's CUDA kernels; this package only
marshals arguments (torch tensors -> device pointers, sizes, the current stream).
"""
from .binding import (  # noqa: F401
    CowaError, Params, Window, lib, lib_path, make_params,
    cowa_fwd, cowa_prefill, cowa_prefill_varlen, cowa_bwd, cowa_decode, cowa_decode_multi, cowa_decode_paged, cowa_decode_multi_workspace_bytes,
    cowa_decode_static, cowa_decode_static_capacity,
    cowa_bwd_workspace_bytes, cowa_bwd_varlen, cowa_bwd_varlen_workspace_bytes,
    cowa_bwd_prefill, cowa_bwd_prefill_workspace_bytes, with_bwd_events, cowa_decode_workspace_bytes,
    cowa_default_windows, cowa_equal_area_windows, cowa_schedule_dump, cowa_tile_counts, cowa_check_device_status,
    cowa_selftest_bounded_wait,
    cowa_status_string, SCHED_FWD, SCHED_BWD, SCHED_DECODE,
)
