"""R-Stitch routing decision at the LM head, B200-native (sm_100a CUDA behind a C ABI).

The Python layer only marshals arguments: every step of the path runs in the kernels of
``librstitch.so``.  There is no CPU or PyTorch fallback; a missing library raises.
"""
from .binding import (  # noqa: F401
    RstitchError, Handle, Alg1State, LatencyModel, Router, RouteOutputs, PreparedCall, PreparedHostCall, route_ex_host, lib, library_path, route, route_ex, route_host, route_static, STATIC_MAX_ROWS, compact, shard_stats, shard_route, SHARD_WORDS, selftest_wait, probe_read_stream, SELFTEST_SITE,
    last_status, workspace_bytes, status_string, path_name,
    TAU_NORMALIZED, SAMPLE, PATH_GEMV, PATH_UMMA,
)
