"""B200-native forward path of Pyramid Sparse Attention: thin ctypes binding over libpisa.so.

Argument marshalling only — every step of the path runs in the library's CUDA kernels.  PyTorch is
used for device memory and streams.  Importing this package does not load the library; the first
call does, and fails loudly if it has not been built (`python -m paper_2609_31093_b200.build`).
"""
from .binding import (  # noqa: F401
    PisaError,
    Params,
    lib,
    pyramid_layout,
    workspace_bytes,
    pisa_build_pyramid,
    pisa_route,
    pisa_route_static,
    route_static_capacity,
    pisa_bsa_fwd,
    pisa_forward,
    pisa_forward_host,
    pisa_forward_packed,
    packed_plan,
    pisa_flat_select,
    pisa_bsa_bwd,
    pisa_bsa_bwd_packed,
    pisa_decode_step,
    pisa_pyramid_regrow,
    read_status,
    debug_wait_timeout,
    DEBUG_BOUNDS,
    set_stage_timing,
    get_stage_ms,
    launch_count,
    get_kernel_ms,
    get_kernel_brackets,
    set_forward_chunks,
    IMPL_AUTO,
    IMPL_SIMT,
    IMPL_TENSOR,
)
