"""Seeded synthetic workloads (data only).

This package produces the key / value / query arrays that both the CUDA path and
the CPU oracle consume.  It contains no arithmetic of the retrieval method: no
distances, no clustering, no attention.
"""
from .workloads import CONFIGS, WorkloadConfig, UnitStream, make_prefill, make_decode_chunk, unit_seed

__all__ = ["CONFIGS", "WorkloadConfig", "UnitStream", "make_prefill", "make_decode_chunk", "unit_seed"]
