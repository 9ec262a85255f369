"""B200-native hot path of ActKV's action-guided KV-cache compression.

`binding` holds the ctypes binding of the C-ABI library (actkv_score / actkv_select /
actkv_compact / actkv_budget), `harness` the torch-side owner of pool, tables and scratch,
`synth` the seeded workload generators.  Nothing is loaded at import time; the CUDA library
is opened on first use and its absence is an error, never a fallback.
"""
__all__ = ["binding", "harness", "synth"]
