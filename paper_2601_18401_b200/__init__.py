"""B200 (sm_100a) span-search + span-attention for N=2 Superlinear attention.

The product is ``libsla.so`` (C interface in ``include/sla.h``); this package holds its CUDA
sources (``csrc/``), the build step (``build.py``), a ctypes binding with the same call names
(``binding.py``) and the seeded synthetic-input generators (``synth.py``).
"""
from .binding import (  # noqa: F401
    Handle, SlaError, SLA_BF16, SLA_F32, SLA_OK, SLA_PER_SPAN, SLA_UNION, load_library, make_layout,
    make_params, sla_attention_tile_stats, sla_decode_shard_attend, sla_decode_shard_merge, sla_decode_shard_search, sla_decode_step, sla_decode_step_static, sla_host_staging_bytes, sla_kernel_launches, sla_kernel_time_ms, sla_set_kernel_timing, sla_layout_t, sla_params_t, sla_poll_status,
    sla_pattern_len_steps, sla_pattern_offsets, sla_probe_l2_read, sla_selftest_canary_trip, sla_selftest_wait_expiry, sla_set_debug_canaries, sla_prefill_host, sla_span_attention, sla_span_attention_gated, sla_span_search, sla_workspace_bytes,
)
