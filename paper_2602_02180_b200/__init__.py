"""STILL intra-layer hybrid attention forward for B200 (sm_100a): Python binding of libstill.so."""
from .binding import (  # noqa: F401
    StillError,
    StillParams,
    device_status,
    host_arena_bytes,
    hybrid_attn_fwd,
    hybrid_attn_fwd_host,
    hybrid_attn_fwd_static,
    hybrid_attn_step,
    last_launch_count,
    profile_collect,
    profile_enable,
    selftest_wait_timeout,
    state_bytes,
    state_layout,
    strerror,
    workspace_bytes,
)
from .build import build_library  # noqa: F401
