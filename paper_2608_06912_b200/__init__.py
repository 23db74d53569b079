"""B200 (sm_100a) LapSum exact-budget soft top-k: CUDA library + thin binding.

The public calls mirror the C ABI of include/lapsum.h one to one.
"""
from .binding import (  # noqa: F401
    PATH_AUTO, PATH_BLOCK, PATH_BRACKET, PATH_FULLSORT, PATH_NAMES, ST_BAND_OVERFLOW, ST_FALLBACK,
    ST_LOOKBACK_TIMEOUT, ST_NO_CROSSING, ST_ROOT_LEFT, ST_ROOT_RIGHT, ST_WIDENED, ST_BAD_BUDGET, LapsumError, Params, Workspace,
    default_params, lapsum_backward, lapsum_debug_bracket, lapsum_debug_sort_pairs, lapsum_forward,
    lapsum_forward_with_bracket, lapsum_launch_count, lapsum_profile_disable, lapsum_profile_enable,
    lapsum_profile_read, KERNELS, lapsum_backward_static, lapsum_backward_scalars, lapsum_forward_backward_host,
    lapsum_describe, lapsum_forward_row_budgets, lapsum_debug_lookback_timeout, lapsum_forward_rows, lapsum_backward_rows, ST_BAD_ALPHA, ST_BOUNDS,
    lapsum_forward_io, lapsum_backward_io, ShardWorkspace, GpuShard, IO_F32, IO_F16, IO_BF16, IO_TORCH, IO_NAMES, lapsum_workspace_bytes, lib, library_path,
)
