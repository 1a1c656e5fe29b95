"""B200-native (sm_100a) implementation of the WeDLM streaming-parallel-decoding step.

The product is the C-ABI shared library built from ``csrc/`` (declared in ``include/wedlm.h``).
This package is the thin Python binding over it: it marshals torch device tensors into raw
pointers and launches on torch's current CUDA stream.  There is no CPU or PyTorch fallback: if
the library has not been built, every call raises.
"""
from .binding import (  # noqa: F401
    WedlmConfig,
    WedlmError,
    DecodeStep,
    config_for,
    to_device,
    library_path,
    load_library,
    make_config,
    wedlm_confidence_commit,
    wedlm_confidence_commit_static,
    wedlm_confidence_workspace_bytes,
    wedlm_dual_stream_attn,
    wedlm_dual_stream_construct,
    wedlm_dual_stream_workspace_bytes,
    wedlm_kv_append,
    wedlm_launch_count,
    wedlm_lmhead_confidence_commit,
    wedlm_lmhead_confidence_workspace_bytes,
    wedlm_profile_next_attn,
    wedlm_reorder,
    wedlm_selftest_wait_expiry,
    wedlm_step_host,
    wedlm_step_host_lmhead,
    wedlm_step_host_lmhead_workspace_bytes,
    wedlm_step_host_workspace_bytes,
    wedlm_strerror,
    wedlm_version,
    wedlm_window_attn,
    wedlm_window_attn_workspace_bytes,
    wedlm_window_refill,
)
