"""B200 (sm_100a) implementation of the per-turn GPU path EFIM leaves to compute:
fused RoPE + paged KV append, append-prefill attention over cached + new keys, and
split-KV paged decode attention.  The work is done by the CUDA library
`libefim.so` (C ABI in include/efim.h); this package only marshals arguments.
"""
from .binding import (  # noqa: F401
    EfimError, Cache, Batch, Rope, load_library, library_path, exported_symbols,
    efim_kv_append, efim_append_prefill_attn, efim_decode_attn,
    efim_prefill_workspace_bytes, efim_decode_workspace_bytes, efim_rope_table_build,
    efim_strerror, efim_version, efim_decode_attn_static, efim_decode_static_scratch_bytes,
    efim_prefill_launch_count, efim_decode_launch_count, Frontend, efim_prefill_plan, efim_decode_step,
    efim_append_prefill_step, efim_selftest_bounded_wait,
)
