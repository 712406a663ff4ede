"""Seeded synthetic inputs shaped like the paper's workloads.

This package holds the workload table and the random input generators only. It contains none of
the method's arithmetic (no attention, no scoring, no eviction) and is the one module that both
the CUDA library's callers and the CPU oracle's callers may share.
"""
from .configs import CONFIGS, Workload, get, scaled  # noqa: F401
from .generators import decode_inputs, prefill_inputs, prompt_lengths  # noqa: F401
