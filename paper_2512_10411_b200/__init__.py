"""SWAA attention hot path for NVIDIA B200 (sm_100a).

``swaa_prefill`` / ``swaa_decode`` and the host-side layer schedule, as a C-ABI
shared library (``csrc/``, ``include/swaa.h``) plus this thin ctypes binding.
The library is loaded on first use; there is no CPU fallback: a missing or
unloadable library raises.
"""
from .binding import (  # noqa: F401
    SwaaError,
    SwaaPolicy,
    decode_num_blocks,
    decode_workspace_size,
    kernel_launch_count,
    prefill_block_shape,
    prefill_tile_needs_mask,
    prefill_tile_range,
    lib_path,
    load_library,
    schedule_fill,
    schedule_is_full,
    schedule_select_fa_layers,
    status_str,
    swaa_decode,
    swaa_decode_paged,
    swaa_decode_partial,
    swaa_decode_combine,
    decode_partial_workspace_size,
    decode_paged_workspace_size,
    swaa_decode_static,
    DECODE_STATIC_SCRATCH_BYTES,
    swaa_lazy_ratio,
    swaa_prefill,
    swaa_prefill_backward,
    prefill_backward_workspace_size,
    swaa_prefill_chunked,
    swaa_prefill_context_parallel,
    swaa_prefill_paged,
    last_device_status,
    trimmed_cache_len,
    trimmed_cache_slot,
)
