"""HashEvict eviction hot path for B200: a thin ctypes binding over the CUDA library (see binding.py)."""
from .binding import (  # noqa: F401
    HE_FLAG_EARLY_INPUTS, HE_FLAG_PACKED_CODES, HE_FLAG_WRITE_SCORES, HashEvictCache, HashEvictError, decode_staging_bytes, device_error_count, hash_keys, lib,
    prefill_phase_events,
    prefill_staging_bytes,
    workspace_bytes,
)
