"""Increasing batch-size schedule of Section 5.2.2 (host arithmetic only).

The batch grows from 262,144 to 1,048,576 examples over the first 7,500 steps: every quarter of that ramp
(1,875 steps) it is raised by 196,608 examples, reaching 1,048,576 at step 7,500 and staying there.  The step
kernels take the batch size of each macro-step as an argument, so a schedule only changes how many microbatches
are accumulated before `finish_macro_batch` and the divisor passed to it.
"""
from __future__ import annotations


def increasing_batch_size(t: int, start: int = 262_144, end: int = 1_048_576, ramp_steps: int = 7_500,
                          increments: int = 4) -> int:
    """Batch size q_t at step t (t counts from 0 or 1 alike: the raises happen at multiples of ramp/increments)."""
    if t < 0:
        raise ValueError("step must be non-negative")
    quarter = ramp_steps // increments
    k = min(increments, t // quarter)
    return start + k * ((end - start) // increments)


def microbatches_for_step(t: int, microbatch: int, **kw) -> int:
    """Number of microbatches of `microbatch` examples that make up q_t (q_t must be a multiple)."""
    q = increasing_batch_size(t, **kw)
    if q % microbatch:
        raise ValueError(f"batch size {q} is not a multiple of the microbatch {microbatch}")
    return q // microbatch
