"""B200-native FlashAttention forward with the Sawtooth Wavefront Reordering K/V scan.

A thin ctypes binding over libsawtooth_attn.so (the C-ABI library built from csrc/).  Every step of
the attention pass runs in the library's CUDA kernels; this package only marshals arguments.  There
is no CPU fallback: without the built library, or without a B200, the calls raise.
"""
from .binding import (  # noqa: F401
    CYCLIC, SAWTOOTH, F16, BF16, TILE_FASTEST, HEAD_FASTEST, PAIR_DEFAULT, PAIR_NONE, PAIR_MIRRORED, PAIR_ADJACENT, LAYOUT_BHND, LAYOUT_BNHD,
    AttnError, Opts, Plan, TraceEntry,
    attn_fwd, attn_fwd_ex, attn_fwd_dynamic, attn_fwd_dynamic_noalloc, attn_dynamic_scratch_bytes, attn_fwd_host, attn_host_groups, attn_query_plan, attn_schedule_trace, attn_dynamic_claim_trace,
    attn_device_status, attn_last_kernel_cycles, attn_status_string, attn_last_error, library_path, load_library,
    forward,
)
