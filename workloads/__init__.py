"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This package only draws random tensors and describes workload shapes.  It holds
none of the method's arithmetic (no attention, no scores, no selection), so both
the CPU oracle and the CUDA path can be fed from it without sharing any logic.
"""
from .synth import (  # noqa: F401
    CONFIGS,
    Workload,
    budgets_for,
    make_decode_inputs,
    make_prompt_inputs,
    ragged_prompt_lengths,
)
