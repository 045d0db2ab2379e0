"""Thin Python binding of the psa C library (``include/psa.h``): argument marshalling only.

Every step of the path runs in the CUDA library.  There is no fallback: if
``libpsa.so`` has not been built, or no CUDA device is present when a kernel is
requested, the call raises.
"""
from .binding import (  # noqa: F401
    PsaError, Plan, PlanInfo, decode, decode_host, decode_static, static_check_status, static_selftest_bounded_wait, append_kv, append_kv_alloc, prefill, sample_tokens, sample_tokens_at, attn_task, library, library_path, status_string, EXPORTED_SYMBOLS,
)
