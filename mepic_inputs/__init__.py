"""Seeded synthetic inputs for the MEPIC hot path.

This package holds input generation only: chunk token ids, request segment
lists, the random bf16 K/V page pool, query vectors and new-row K/V for
prefill.  It contains none of the method's arithmetic (no table construction,
no rotary embedding, no attention), so both the CPU oracle's tests and the
CUDA path's tests may draw their inputs from it without sharing code that is
under test.
"""
from .bf16 import f32_to_bf16_bits, bf16_bits_to_f32, bf16_bits_to_f64
from .workloads import (Workload, Request, PrefillRows, make_workload,
                        make_custom, CONFIG_NAMES)

__all__ = ["f32_to_bf16_bits", "bf16_bits_to_f32", "bf16_bits_to_f64",
           "Workload", "Request", "PrefillRows", "make_workload",
           "make_custom", "CONFIG_NAMES"]
