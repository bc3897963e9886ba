"""Seeded synthetic LVLM-cache workloads (input generators only: no AirCache arithmetic lives here).

The same generator feeds the CPU oracle and the CUDA library.  Every large tensor is a pure
function of (seed, tensor id, layer, sequence, element index) built from integer hashing, a
table lookup and at most one fp32 add, so that the CPU and the GPU produce identical bf16 bits
and any slice can be regenerated on its own.
"""
from .synth import (CONFIGS, Workload, decode_queries, full_cache, normal_table, plan, window_queries)

__all__ = ["CONFIGS", "Workload", "decode_queries", "full_cache", "normal_table", "plan", "window_queries"]
