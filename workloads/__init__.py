"""Seeded synthetic inputs shared by the tests, the benchmark and the oracle's callers.

This package holds no arithmetic of the method itself: it only describes the
five workload shapes and draws Q/K/V tensors (plus the positional structure a
model would already have applied to them).
"""
from .configs import Workload, CONFIGS, get_config, alibi_slopes
from .synth import make_prompt, make_step, unit_list, sample_units

__all__ = ["Workload", "CONFIGS", "get_config", "alibi_slopes",
           "make_prompt", "make_step", "unit_list", "sample_units"]
