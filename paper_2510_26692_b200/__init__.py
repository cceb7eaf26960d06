"""B200-native KDA (Kimi Delta Attention) hot path: chunkwise prefill and recurrent decode.

The product is the CUDA library behind the C ABI declared in ``include/kda.h``; this package holds
its sources (``csrc/``), the build step (``build``) and a thin ctypes binding with the same
entry-point names (``api``).  ``inputs`` draws the seeded synthetic workloads.  The library is
loaded on first use and there is no fallback path: a missing ``libkda_b200.so`` raises.
"""
from .api import (  # noqa: F401
    KDA_BF16, KDA_F32, KdaError, kda_check_status, kda_chunk_bwd, kda_chunk_bwd_workspace_bytes, kda_chunk_fwd, kda_chunk_fwd_host,
    kda_chunk_fwd_host_workspace_bytes, kda_chunk_fwd_min_workspace_bytes, kda_chunk_fwd_static, kda_chunk_fwd_static_check_status, kda_chunk_fwd_static_max_bytes,
    kda_chunk_fwd_workspace_bytes, kda_decode_multi, kda_decode_step, kda_dplr_chunk_fwd, kda_dplr_chunk_fwd_min_workspace_bytes, kda_dplr_chunk_fwd_workspace_bytes, kda_decode_step_host,
    kda_decode_step_host_workspace_bytes, kda_last_error, kda_layer_decode_step, kda_layer_fwd, kda_layer_fwd_min_workspace_bytes, kda_layer_fwd_workspace_bytes, kda_layer_set_fused_output, kda_launch_count, kda_profile_enable, kda_profile_read, kda_selftest_wait_timeout, kda_set_chunk_path, kda_version,
    library_path,
)
