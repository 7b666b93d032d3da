"""Per-step scalars of the paper's training recipe, for ``asyncmesh_step_ex``.

The library takes the EMA coefficient and the learning rate of a step as plain
numbers; these helpers produce the sequences the paper trains with.  Host logic
only, no state.
"""
from __future__ import annotations

import math


def ema_coefficient(t: int, total_steps: int, start: float = 0.5, end: float = 0.01,
                    hold: int = 1000) -> float:
    """lambda_t of Eq. "ema" as scheduled in Section 3.3: ``start`` for the first
    ``hold`` iterations, then a cosine decay that reaches ``end`` at
    ``total_steps``.  ``t`` counts steps from 1."""
    if t <= hold or total_steps <= hold:
        return start
    x = min(1.0, (t - hold) / float(total_steps - hold))
    return end + 0.5 * (start - end) * (1.0 + math.cos(math.pi * x))


def learning_rate(t: int, total_steps: int, peak: float = 3e-4, floor: float = 3e-5,
                  warmup: int = 3000, start: float = 1e-7) -> float:
    """The learning-rate schedule of Appendix B.1: linear warm-up from ``start``
    to ``peak`` over ``warmup`` iterations, then a cosine decay to ``floor`` at
    ``total_steps``.  ``t`` counts steps from 1."""
    if t <= warmup:
        return start + (peak - start) * (t / float(warmup))
    if total_steps <= warmup:
        return peak
    x = min(1.0, (t - warmup) / float(total_steps - warmup))
    return floor + 0.5 * (peak - floor) * (1.0 + math.cos(math.pi * x))
