"""B200-native batched evaluation of the hybrid offline-online scheduler (arXiv 2502.15763).

The work is done by libhos.so (hand-written CUDA for sm_100a behind a C ABI, see
include/hos.h).  This package is the thin Python binding: it marshals torch
device tensors into the C calls and nothing else.  There is no CPU fallback:
calling a compute entry point without the library or without a CUDA device
raises.
"""
from .binding import (  # noqa: F401
    CLIENT_RESULT_DTYPE, ITER_REC_DTYPE, LB_DTYPE, LS_MOVE_DTYPE, SIM_RESULT_DTYPE,
    HOS_QUEUE_FCFS, HOS_QUEUE_SORTED, HOS_ST_INVALID, HOS_ST_LIMIT, HOS_ST_RANGE, HOS_ST_TRACE,
    HosError, exported_symbols, hos_debug_bounds_violations, hos_local_search, hos_lower_bound, hos_lower_bound_static, hos_offline_pack,
    hos_online_simulate, hos_online_simulate_steal, hos_set_launch_hook, hos_strerror, hos_trace_fill, hos_trace_offsets, lib, lib_path,
)
