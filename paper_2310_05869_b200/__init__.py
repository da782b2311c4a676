"""B200-native HyperAttention forward (arXiv 2310.05869): thin binding over libhyperattn.so."""
from .binding import (  # noqa: F401
    HyperAttnError,
    alpha,
    backward,
    forward,
    forward_host,
    get_projections,
    last_device_status,
    lib,
    profile_enable,
    profile_read,
    profile_reset,
    release,
    sortlsh_noalloc,
    version,
    workspace_bytes,
)
