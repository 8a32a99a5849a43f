"""B200-native exhaustive search over fused-attention dataflow mappings (MMEE hot path).

The product is the CUDA library `libmmee.so` (sources under csrc/, C ABI in include/mmee.h);
`binding` exposes its entry points under the same names.
"""
from .binding import (  # noqa: F401
    ERR_ARG, ERR_CHECK, ERR_CUDA, ERR_NO_FEASIBLE, ERR_OVERFLOW, ERR_QUANTUM, ERR_RANGE, NO_INDEX, OK,
    MmeeError, Result, library, mmee_alu_peak, mmee_create, mmee_decode, mmee_destroy, mmee_dump_keys, mmee_eval, mmee_filter_flags,
    mmee_kernel_timing, mmee_last_search_stats, mmee_num_candidates, mmee_pareto_front, mmee_pareto_front_bs_da, mmee_num_rows, mmee_num_tilings,
    mmee_query_vector, mmee_recompute_flag, mmee_row_pruning_keep, mmee_search, mmee_search_host, mmee_search_shapes, mmee_search_static, mmee_solve_host, read_results, result_buffer,
)
