"""Seeded synthetic inputs for the EFIM append-prefill / paged-decode path.

This package holds only input generation: bf16 bit conversion of random
draws, a counter-based fill for the paged KV pools, ragged length draws and
block tables.  It contains none of the method's arithmetic (no RoPE, no
softmax, no attention) and imports neither the CPU oracle nor the CUDA
library; both are fed from here with identical bytes.
"""
from .bf16 import f32_to_bf16_bits, bf16_bits_to_f32
from .pool import pool_bits_np, pool_fill_torch
from .workloads import Workload, make_workload, WORKLOAD_NAMES

__all__ = [
    "f32_to_bf16_bits", "bf16_bits_to_f32", "pool_bits_np", "pool_fill_torch",
    "Workload", "make_workload", "WORKLOAD_NAMES",
]
from .sessions import token_tables, infill_sessions, TOK_P, TOK_S, TOK_M  # noqa: F401,E402
